// Per-Gaussian kernels: projection with fused appearance decode (forward and backward) and the
// separate-pass appearance kernels.  One thread per Gaussian; the parameter rows of the explicit models
// (SH coefficients, Spherical Voronoi sites) and their gradients move through per-warp shared-memory
// slabs so that global accesses stay coalesced; the neural decoder runs on warp-level tensor-core tiles
// with its weights in shared memory.
#include <float.h>
#include <stdio.h>
#include <string.h>

#include "gs_device.cuh"
#include "gs_mlp_mma.cuh"

namespace gs {
namespace {

constexpr int kBlock = 128;
constexpr int kWarps = kBlock / 32;
// Floats per Gaussian of the explicit models' parameter rows: 45 SH coefficients (bands 1..3, RGB) or the
// 7 x 7 raw site parameters of Spherical Voronoi.  Both are odd, so a lane reading its own row in a
// warp's shared-memory slab of 32 rows meets no bank conflict.
template <int APP> struct RowOf { static constexpr int value = APP == GS_APP_SV ? GS_SV_ROW : GS_SH_REST; };
template <int APP> struct SlabOf { static constexpr int value = 32 * RowOf<APP>::value; };
template <int APP> struct Explicit { static constexpr bool value = APP == GS_APP_SH || APP == GS_APP_SV; };
// The neural model in either precision of its decoder's products: fp16 operands split into two halves (results as
// accurate as fp32 FMAs, the default), or plain fp16 operands as the paper runs it (kAppNeuralHalf).
template <int APP> struct IsNeural { static constexpr bool value = APP == GS_APP_NEURAL || APP == kAppNeuralHalf; };
template <int APP> struct Split { static constexpr bool value = APP != kAppNeuralHalf; };
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ bool finite_f(float x) { return fabsf(x) <= FLT_MAX; }

// ---- warp-cooperative row movement ----------------------------------------------------------
template <int kRow>
__device__ __forceinline__ void warp_load_rows(const float *g, int64_t row0, int64_t n, float *slab,
                                               int lane) {
  const int rows = (int)min((int64_t)32, n - row0);
  const int total = rows * kRow;
  const float *src = g + row0 * kRow;     // row0 is a multiple of 32 => 16-byte aligned
  const int nv = total >> 2;
  for (int k = lane; k < nv; k += 32) reinterpret_cast<float4 *>(slab)[k] = __ldg(reinterpret_cast<const float4 *>(src) + k);
  for (int k = (nv << 2) + lane; k < total; k += 32) slab[k] = __ldg(src + k);
  __syncwarp();
}

template <int kRow>
__device__ __forceinline__ void warp_store_rows(float *g, int64_t row0, int64_t n, const float *slab,
                                                int lane) {
  __syncwarp();
  const int rows = (int)min((int64_t)32, n - row0);
  const int total = rows * kRow;
  float *dst = g + row0 * kRow;
  const int nv = total >> 2;
  for (int k = lane; k < nv; k += 32) reinterpret_cast<float4 *>(dst)[k] = reinterpret_cast<const float4 *>(slab)[k];
  for (int k = (nv << 2) + lane; k < total; k += 32) dst[k] = slab[k];
  __syncwarp();
}

// ---- 1D bulk copies (tensor memory accelerator) with bounded waits ------------------------------------------
// load(): one lane arms the warp's mbarrier with the byte count and starts the copy; wait(): every lane polls the
// barrier's phase, at most about a second in all; store(): shared -> global as a bulk group of the issuing lane.
namespace bulk {
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void barrier_init(uint32_t bar) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 20); ++it) {   // each try sleeps at most about a microsecond: the wait ends within a second
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void store(void *dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void wait_stores_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void wait_stores_done() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_generic_writes() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
}  // namespace bulk

// ---- appearance: SH -------------------------------------------------------------------------
// colour = max(0, c0 + 0.5 + sum_k Y_k(d) c_k); row = this Gaussian's 45 coefficients in smem.
__device__ __forceinline__ void sh_decode(const float *row, const float base[3], float dx, float dy,
                                          float dz, int deg, float pre[3]) {
  float Y[16];
  sh_basis(dx, dy, dz, Y);
  const int na = (deg + 1) * (deg + 1);
  float r = base[0] + 0.5f, g = base[1] + 0.5f, b = base[2] + 0.5f;
#pragma unroll
  for (int k = 1; k < 16; ++k) {
    if (k < na) {
      r = fmaf(Y[k], row[3 * (k - 1) + 0], r);
      g = fmaf(Y[k], row[3 * (k - 1) + 1], g);
      b = fmaf(Y[k], row[3 * (k - 1) + 2], b);
    }
  }
  pre[0] = r; pre[1] = g; pre[2] = b;
}

// Backward of the SH decode.  gp = dL/d(pre-activation) (already masked by the ReLU).  Writes the
// coefficient gradients over `row` in place (row holds the coefficients on entry) and returns
// dL/dd.
__device__ __forceinline__ void sh_backward(float *row, const float gp[3], float dx, float dy, float dz,
                                            int deg, float gd[3]) {
  float Y[16];
  sh_basis(dx, dy, dz, Y);
  const int na = (deg + 1) * (deg + 1);
  float gx = 0.f, gy = 0.f, gz = 0.f;
#pragma unroll
  for (int k = 1; k < 16; ++k) {
    float *c = row + 3 * (k - 1);
    if (k < na) {
      const float w = c[0] * gp[0] + c[1] * gp[1] + c[2] * gp[2];
      sh_grad_acc(k, dx, dy, dz, w, gx, gy, gz);
      c[0] = Y[k] * gp[0]; c[1] = Y[k] * gp[1]; c[2] = Y[k] * gp[2];
    } else {
      c[0] = 0.f; c[1] = 0.f; c[2] = 0.f;
    }
  }
  gd[0] = gx; gd[1] = gy; gd[2] = gz;
}

// ---- appearance: Spherical Voronoi (Eq. 3) ---------------------------------------------------
// row = this Gaussian's 7 sites x (a_r, a_g, a_b, s_x, s_y, s_z, t) in shared memory.  s = raw / |raw|,
// tau = exp(t), rho = |s - d|, A = sum_i softmax_i(-tau_i rho_i) a_i.  One pass over the sites with a running
// maximum (App. B): when a larger logit turns up, what has been summed so far is rescaled.
__device__ __forceinline__ float sv_logit(const float *p, float dx, float dy, float dz) {
  const float inv = rsqrtf(fmaf(p[3], p[3], fmaf(p[4], p[4], p[5] * p[5])));
  const float ex = fmaf(p[3], inv, -dx), ey = fmaf(p[4], inv, -dy), ez = fmaf(p[5], inv, -dz);
  return -expf(p[6]) * sqrtf(fmaf(ex, ex, fmaf(ey, ey, ez * ez)));
}
__device__ __forceinline__ void sv_decode(const float *row, float dx, float dy, float dz, float A[3], float &mx, float &z) {
  mx = -FLT_MAX; z = 0.f;
  float r = 0.f, g = 0.f, b = 0.f;
#pragma unroll
  for (int i = 0; i < GS_SV_SITES; ++i) {
    const float *p = row + 7 * i;
    const float l = sv_logit(p, dx, dy, dz);
    if (l > mx) { const float sc = expf(mx - l); z *= sc; r *= sc; g *= sc; b *= sc; mx = l; }
    const float e = expf(l - mx);
    z += e; r = fmaf(e, p[0], r); g = fmaf(e, p[1], g); b = fmaf(e, p[2], b);
  }
  const float iz = 1.f / z;
  A[0] = r * iz; A[1] = g * iz; A[2] = b * iz;
}
// Backward, second pass (the first is sv_decode, which leaves A, the maximum and the normaliser): writes the
// site gradients over `row` in place and returns dL/dd.  gA = dL/dA.
__device__ __forceinline__ void sv_backward(float *row, const float gA[3], const float A[3], float mx, float z, float dx,
                                            float dy, float dz, float gd[3]) {
  const float Ag = A[0] * gA[0] + A[1] * gA[1] + A[2] * gA[2], iz = 1.f / z;
  float gx = 0.f, gy = 0.f, gz = 0.f;
#pragma unroll
  for (int i = 0; i < GS_SV_SITES; ++i) {
    float *p = row + 7 * i;
    const float a0 = p[0], a1 = p[1], a2 = p[2];
    const float len2 = fmaf(p[3], p[3], fmaf(p[4], p[4], p[5] * p[5]));
    const float inv = rsqrtf(len2);
    const float sx = p[3] * inv, sy = p[4] * inv, sz = p[5] * inv;
    const float ex = sx - dx, ey = sy - dy, ez = sz - dz;
    const float rho = sqrtf(fmaf(ex, ex, fmaf(ey, ey, ez * ez)));
    const float tau = expf(p[6]);
    const float w = expf(-tau * rho - mx) * iz;
    const float g_logit = w * (a0 * gA[0] + a1 * gA[1] + a2 * gA[2] - Ag);
    const float g_rho = -tau * g_logit;
    const float ir = rho > 0.f ? 1.f / rho : 0.f;      // no gradient of the distance where it vanishes
    const float ux = g_rho * ex * ir, uy = g_rho * ey * ir, uz = g_rho * ez * ir;   // dL/ds
    gx -= ux; gy -= uy; gz -= uz;
    const float dot = ux * sx + uy * sy + uz * sz;     // through the normalisation
    p[0] = w * gA[0]; p[1] = w * gA[1]; p[2] = w * gA[2];
    p[3] = (ux - dot * sx) * inv; p[4] = (uy - dot * sy) * inv; p[5] = (uz - dot * sz) * inv;
    p[6] = -rho * g_logit * tau;
  }
  gd[0] = gx; gd[1] = gy; gd[2] = gz;
}

// ---- the two explicit models behind one pair of calls -----------------------------------------
struct SvCarry { float A[3], mx, z; };   // what the SV backward needs from its first pass
template <int APP>
__device__ __forceinline__ void explicit_pre(const float *row, const float base[3], float dx, float dy, float dz, int deg,
                                             float pre[3], SvCarry &cy) {
  if (APP == GS_APP_SV) {
    cy.A[0] = cy.A[1] = cy.A[2] = 0.f; cy.mx = 0.f; cy.z = 1.f;
    if (deg > 0) sv_decode(row, dx, dy, dz, cy.A, cy.mx, cy.z);
    pre[0] = base[0] + 0.5f + cy.A[0]; pre[1] = base[1] + 0.5f + cy.A[1]; pre[2] = base[2] + 0.5f + cy.A[2];
  } else {
    sh_decode(row, base, dx, dy, dz, deg, pre);
  }
}
template <int APP>
__device__ __forceinline__ void explicit_bwd(float *row, const float gp[3], float dx, float dy, float dz, int deg,
                                             const SvCarry &cy, float gd[3]) {
  if (APP == GS_APP_SV) {
    if (deg > 0) {
      sv_backward(row, gp, cy.A, cy.mx, cy.z, dx, dy, dz, gd);
    } else {
#pragma unroll
      for (int k = 0; k < GS_SV_ROW; ++k) row[k] = 0.f;
      gd[0] = gd[1] = gd[2] = 0.f;
    }
  } else {
    sh_backward(row, gp, dx, dy, dz, deg, gd);
  }
}

// ---- appearance: neural ---------------------------------------------------------------------
// Forward-only staging of the tensor-core decoder: the leading members of mlp::WarpStage.
struct __align__(16) StageFwd {
  uint32_t xhi[32 * mlp::kXStride];
  uint32_t xlo[32 * mlp::kXStride];
  float y[32 * 4];
};

// Whole-warp decode: every lane passes its Gaussian's inputs (zeros if it has none) and gets the
// tanh-bounded residual A back.  All 32 lanes must call it.
template <bool kSplit, class Stage>
__device__ __forceinline__ void decode_warp(const mlp::FwdFrags &F, Stage &S, int lane, const float x[32],
                                            mlp::Activations &act, float A[3]) {
  mlp::stage_inputs<kSplit>(x, S, lane);
  mlp::forward_warp<kSplit>(F, S, lane, act);
  const float4 y = *reinterpret_cast<const float4 *>(S.y + lane * 4);
  A[0] = tanh_fast(y.x); A[1] = tanh_fast(y.y); A[2] = tanh_fast(y.z);
}

// Whole-warp backward of the decoder.  `has`: this lane owns a Gaussian (inputs x, direction d, base
// colour, dL/dcolour gcol); lanes without one pass zeros.  Returns the colour gradient through the activation
// gp, dL/df and dL/dd of the lane's Gaussian and advances the warp's weight-gradient fragments.
template <bool kSplit>
__device__ __forceinline__ void decode_backward_warp(const mlp::Weights &W, mlp::WarpStage &S, int lane, bool has,
                                                     const float x[32], float dx, float dy, float dz, int deg, int cact,
                                                     const float base[3], const float gcol[3], mlp::WeightGrad &dW,
                                                     float gp[3], float gf[8], float gd[3]) {
  mlp::Activations act;
  float A[3];
  {
    const mlp::FwdFrags F = mlp::load_fwd_frags(W.w, lane);   // out of shared memory, every trip: the registers are needed elsewhere
    decode_warp<kSplit>(F, S, lane, x, act, A);
  }
  float gy[3];
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    gp[c] = has ? color_act_grad_z(cact, base[c] + 0.5f + A[c]) * gcol[c] : 0.f;
    gy[c] = gp[c] * (1.f - A[c] * A[c]);
  }
  *reinterpret_cast<float4 *>(S.y + lane * 4) = make_float4(gy[0], gy[1], gy[2], 0.f);
  mlp::backward_warp<kSplit>(W, S, lane, act, dW);
  const float4 f0 = *reinterpret_cast<const float4 *>(S.gf + lane * 8), f1 = *reinterpret_cast<const float4 *>(S.gf + lane * 8 + 4);
  gf[0] = f0.x; gf[1] = f0.y; gf[2] = f0.z; gf[3] = f0.w; gf[4] = f1.x; gf[5] = f1.y; gf[6] = f1.z; gf[7] = f1.w;
  float gx[16];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 v = *reinterpret_cast<const float4 *>(S.gx + lane * mlp::kGxStride + 4 * q);
    gx[4 * q] = v.x; gx[4 * q + 1] = v.y; gx[4 * q + 2] = v.z; gx[4 * q + 3] = v.w;
  }
  const int na = (deg + 1) * (deg + 1);
  float ax = 0.f, ay = 0.f, az = 0.f;
#pragma unroll
  for (int k = 1; k < 16; ++k)
    if (k < na) sh_grad_acc(k, dx, dy, dz, gx[k], ax, ay, az);
  gd[0] = ax; gd[1] = ay; gd[2] = az;
  __syncwarp();
}

// Sum the warps' weight-gradient fragments and write this block's partial [816].  sPart
// ([kWarps][816] floats) may alias the warps' staging areas.
__device__ __forceinline__ void weight_grad_flush(const mlp::WeightGrad &dW, float *sPart, float *partial_out, int tid) {
  __syncthreads();
  mlp::store_weight_grad(dW, sPart + (tid >> 5) * GS_MLP_WEIGHTS, tid & 31);
  __syncthreads();
  for (int k = tid; k < GS_MLP_WEIGHTS; k += kBlock) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) s += sPart[w * GS_MLP_WEIGHTS + k];
    partial_out[k] = s;
  }
}

// Compiler-only fence at the top of the persistent loops: keeps loads of loop-invariant shared
// memory from being hoisted out of the loop into hundreds of live registers.
__device__ __forceinline__ void reload_fence() { asm volatile("" ::: "memory"); }

// Deterministic final reduction of the per-block partials: 32 weights per CTA, the rows shared out over
// sixteen groups of threads (each sums every sixteenth row, in order, four loads in flight), the sixteen sums added
// in a fixed order.
constexpr int kReduceGroups = 16;
__global__ void __launch_bounds__(32 * kReduceGroups) k_wgrad_reduce(const float *__restrict__ partials, int nblocks,
                                                                    float *__restrict__ out) {
  __shared__ float s_part[kReduceGroups][32];
  const int k = blockIdx.x * 32 + threadIdx.x, grp = threadIdx.y;
  float s = 0.f;
  if (k < GS_MLP_WEIGHTS) {
    int b = grp;
    for (; b + 3 * kReduceGroups < nblocks; b += 4 * kReduceGroups) {
      const float p0 = partials[(size_t)b * GS_MLP_WEIGHTS + k], p1 = partials[(size_t)(b + kReduceGroups) * GS_MLP_WEIGHTS + k],
                  p2 = partials[(size_t)(b + 2 * kReduceGroups) * GS_MLP_WEIGHTS + k], p3 = partials[(size_t)(b + 3 * kReduceGroups) * GS_MLP_WEIGHTS + k];
      s += p0; s += p1; s += p2; s += p3;
    }
    for (; b < nblocks; b += kReduceGroups) s += partials[(size_t)b * GS_MLP_WEIGHTS + k];
  }
  s_part[grp][threadIdx.x] = s;
  __syncthreads();
  if (grp == 0 && k < GS_MLP_WEIGHTS) {
    float t = 0.f;
#pragma unroll
    for (int q = 0; q < kReduceGroups; ++q) t += s_part[q][threadIdx.x];
    out[k] = t;
  }
}
inline void launch_wgrad_reduce(const float *partials, int nblocks, float *out, cudaStream_t st) {
  k_wgrad_reduce<<<(GS_MLP_WEIGHTS + 31) / 32, dim3(32, kReduceGroups), 0, st>>>(partials, nblocks, out);
}

// ---- projection -----------------------------------------------------------------------------
struct Geo {
  bool valid;
  float u, v, A, B, C, o, ex, ey, tau;   // (A, B, C) = (l11, l21, l22), the Cholesky factor of the conic
  uint32_t zbits;
  float dirx, diry, dirz;
};

__device__ __forceinline__ void quat_rot(float r, float x, float y, float z, float R[9]) {
  R[0] = 1.f - 2.f * (y * y + z * z); R[1] = 2.f * (x * y - r * z); R[2] = 2.f * (x * z + r * y);
  R[3] = 2.f * (x * y + r * z); R[4] = 1.f - 2.f * (x * x + z * z); R[5] = 2.f * (y * z - r * x);
  R[6] = 2.f * (x * z - r * y); R[7] = 2.f * (y * z + r * x); R[8] = 1.f - 2.f * (x * x + y * y);
}

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// det(N N^T + 0.3 I) without the cancellation of a*c - b*b for elongated splats: by Lagrange's
// identity |N0|^2 |N1|^2 - (N0.N1)^2 = |N0 x N1|^2, so det = |N0 x N1|^2 + 0.3 (|N0|^2 + |N1|^2) + 0.09.
__device__ __forceinline__ float cov_det(const float N[6], float a, float c) {
  const float cx = N[1] * N[5] - N[2] * N[4], cy = N[2] * N[3] - N[0] * N[5], cz = N[0] * N[4] - N[1] * N[3];
  return cx * cx + cy * cy + cz * cz + kDilation * ((a - kDilation) + (c - kDilation)) + kDilation * kDilation;
}

// Everything the backward needs again is recomputed there; this is the forward only.
__device__ __forceinline__ Geo project(const float mu[3], const float ls[3], const float q[4],
                                       float logit, const CamDev &cam) {
  Geo g;
  g.valid = false;
  g.zbits = 0xffffffffu;
  bool fin = finite_f(logit);
#pragma unroll
  for (int k = 0; k < 3; ++k) fin = fin && finite_f(mu[k]) && finite_f(ls[k]);
#pragma unroll
  for (int k = 0; k < 4; ++k) fin = fin && finite_f(q[k]);
  if (!fin) return g;
  // the depth key: one fp32 FMA chain, identical bits on any IEEE machine
  const float z32 = __fmaf_rn(cam.R[8], mu[2], __fmaf_rn(cam.R[7], mu[1], __fmaf_rn(cam.R[6], mu[0], cam.t[2])));
  if (!(z32 >= cam.near_plane) || !(z32 <= cam.far_plane)) return g;
  // The values that leave this function are compared with the oracle's within 1e-5-ish relative bounds; the
  // integers of the tile stage are derived from the STORED values by operations that are rounded correctly
  // (tile_rect, TileSpans).  So here the fast forms of division, square root and exponential do (a few ulp).
  const float o = 1.f / (1.f + expf(-logit));   // accurate: tau = 2 ln(255 o) magnifies its error where o is near 1/255
  if (o < kAlphaMin) return g;
  const float qn2 = q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3];
  if (!(qn2 > 0.f)) return g;
  const float qi = rsqrtf(qn2);
  float R[9];
  quat_rot(q[0] * qi, q[1] * qi, q[2] * qi, q[3] * qi, R);
  const float s0 = __expf(ls[0]), s1 = __expf(ls[1]), s2 = __expf(ls[2]);
  float M[9];
#pragma unroll
  for (int r = 0; r < 3; ++r) { M[3 * r] = R[3 * r] * s0; M[3 * r + 1] = R[3 * r + 1] * s1; M[3 * r + 2] = R[3 * r + 2] * s2; }
  const float tx = cam.R[0] * mu[0] + cam.R[1] * mu[1] + cam.R[2] * mu[2] + cam.t[0];
  const float ty = cam.R[3] * mu[0] + cam.R[4] * mu[1] + cam.R[5] * mu[2] + cam.t[1];
  const float tz = cam.R[6] * mu[0] + cam.R[7] * mu[1] + cam.R[8] * mu[2] + cam.t[2];
  const float iz = __fdividef(1.f, tz);
  const float rx = tx * iz, ry = ty * iz;
  const float txc = tz * fminf(cam.limx, fmaxf(-cam.limx, rx));
  const float tyc = tz * fminf(cam.limy, fmaxf(-cam.limy, ry));
  const float j00 = cam.fx * iz, j02 = -cam.fx * txc * iz * iz;
  const float j11 = cam.fy * iz, j12 = -cam.fy * tyc * iz * iz;
  // T = J R_c (2x3), then N = T M (2x3): cov = N N^T + 0.3 I
  float T[6];
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    T[c] = j00 * cam.R[c] + j02 * cam.R[6 + c];
    T[3 + c] = j11 * cam.R[3 + c] + j12 * cam.R[6 + c];
  }
  float N[6];
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int c = 0; c < 3; ++c) N[3 * r + c] = T[3 * r] * M[c] + T[3 * r + 1] * M[3 + c] + T[3 * r + 2] * M[6 + c];
  const float a = N[0] * N[0] + N[1] * N[1] + N[2] * N[2] + kDilation;
  const float b = N[0] * N[3] + N[1] * N[4] + N[2] * N[5];
  const float c = N[3] * N[3] + N[4] * N[4] + N[5] * N[5] + kDilation;
  const float det = cov_det(N, a, c);
  if (!(det > 0.f) || !finite_f(det)) return g;
  const float tau = footprint_tau(o);
  const float ex = __fmul_rn(sqrt_approx(tau * a), kExtentPad), ey = __fmul_rn(sqrt_approx(tau * c), kExtentPad);
  const float u = fmaf(cam.fx, rx, cam.cx), v = fmaf(cam.fy, ry, cam.cy);
  if (!finite_f(u) || !finite_f(v) || !finite_f(ex) || !finite_f(ey)) return g;
  g.valid = true;
  g.zbits = __float_as_uint(z32);
  // Cholesky factor of the conic Q = cov^-1 = L L^T, straight from the covariance entries (no
  // cancellation even for needle-like splats): l22 = 1/sqrt(c), l11 = sqrt(c/det), l21 = -b/sqrt(c det)
  const float isd = rsqrtf(det), l22 = rsqrtf(c);
  g.u = u; g.v = v; g.A = c * l22 * isd; g.B = -b * l22 * isd; g.C = l22; g.o = o; g.ex = ex; g.ey = ey; g.tau = tau;
  const float vx = mu[0] - cam.oc[0], vy = mu[1] - cam.oc[1], vz = mu[2] - cam.oc[2];
  const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
  g.dirx = vx * vi; g.diry = vy * vi; g.dirz = vz * vi;
  return g;
}

// Tile rectangle of the box [u-ex, u+ex] x [v-ey, v+ey] over pixel centres.  One rounding per
// operation, no contraction, so that the same integers come out of any IEEE fp32 evaluation.
__device__ __forceinline__ bool tile_rect(float u, float v, float ex, float ey, const CamDev &cam,
                                          int r[4]) {
  const float i0 = ceilf(__fsub_rn(__fsub_rn(u, ex), 0.5f)), i1 = floorf(__fsub_rn(__fadd_rn(u, ex), 0.5f));
  const float j0 = ceilf(__fsub_rn(__fsub_rn(v, ey), 0.5f)), j1 = floorf(__fsub_rn(__fadd_rn(v, ey), 0.5f));
  const bool empty = !(i0 <= i1 && j0 <= j1) || i1 < 0.f || j1 < 0.f || i0 > (float)(cam.W - 1) || j0 > (float)(cam.H - 1);
  if (empty) { r[0] = r[1] = r[2] = r[3] = 0; return false; }
  const int pi0 = (int)fmaxf(i0, 0.f), pi1 = (int)fminf(i1, (float)(cam.W - 1));
  const int pj0 = (int)fmaxf(j0, 0.f), pj1 = (int)fminf(j1, (float)(cam.H - 1));
  r[0] = pi0 >> 4; r[1] = pj0 >> 4; r[2] = (pi1 >> 4) + 1; r[3] = (pj1 >> 4) + 1;
  return true;
}

__device__ __forceinline__ void load3(const float *p, int64_t i, float v[3]) {
  v[0] = __ldg(p + 3 * i); v[1] = __ldg(p + 3 * i + 1); v[2] = __ldg(p + 3 * i + 2);
}

// Per-warp shared memory of the cooperative tile-row evaluation: span parameters, rectangle and cell masks of the 32
// owners, and the list of (owner << 8 | row) pairs.
struct RowStage {
  float par[32][8];
  int4 geo[32];
  uint32_t mask[32][9];
  uint32_t tiles[32];
  unsigned short list[32 * 12];
};

template <int APP>
__global__ void __launch_bounds__(kBlock) k_preprocess_fwd(PreprocessArgs a, CamDev cam) {
  dependency_wait();
  __shared__ __align__(16) RowStage sRows[kWarps];
  __shared__ __align__(16) float sData[Explicit<APP>::value ? kWarps * SlabOf<APP>::value : 4];
  __shared__ __align__(16) unsigned char sNN[IsNeural<APP>::value ? kWarps * sizeof(StageFwd) : 16];
  StageFwd *sStage = reinterpret_cast<StageFwd *>(sNN);   // unused for SH
  __shared__ unsigned int sPairs[kWarps];
  __shared__ unsigned long long sBar[kWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t i = (int64_t)blockIdx.x * kBlock + tid;
  const int64_t row0 = (int64_t)blockIdx.x * kBlock + warp * 32;
  const bool in = i < a.n;
  Geo g;
  g.valid = false;
  int rect[4] = {0, 0, 0, 0};
  bool vis = false;
  float mu[3] = {0.f, 0.f, 0.f}, ls[3] = {0.f, 0.f, 0.f}, q[4] = {1.f, 0.f, 0.f, 0.f}, logit = 0.f;
  if (in) {
    load3(a.means, i, mu);
    load3(a.log_scales, i, ls);
    const float4 q4 = __ldg(reinterpret_cast<const float4 *>(a.quats) + i);
    q[0] = q4.x; q[1] = q4.y; q[2] = q4.z; q[3] = q4.w;
    logit = __ldg(a.logits + i);
  }
  // SH / Spherical Voronoi: the warp's slab of parameter rows is one contiguous piece of memory.  Unless the depth
  // test already culls the whole warp, a bulk copy brings it in while the projection below runs (a ragged last
  // warp uses plain loads further down).
  bool slab_by_copy = false;
  if (Explicit<APP>::value && a.deg > 0 && row0 + 32 <= a.n) {
    const float z = __fmaf_rn(cam.R[8], mu[2], __fmaf_rn(cam.R[7], mu[1], __fmaf_rn(cam.R[6], mu[0], cam.t[2])));
    slab_by_copy = __any_sync(kFull, z >= cam.near_plane && z <= cam.far_plane);
    if (slab_by_copy && lane == 0) {
      const uint32_t bar = bulk::smem_addr(sBar + warp);
      bulk::barrier_init(bar);
      bulk::fence_barrier_init();
      bulk::load(bulk::smem_addr(sData + warp * SlabOf<APP>::value), a.sh_rest + row0 * RowOf<APP>::value,
                 SlabOf<APP>::value * sizeof(float), bar);
    }
  }
  if (in) {
    g = project(mu, ls, q, logit, cam);
    if (g.valid) vis = tile_rect(g.u, g.v, g.ex, g.ey, cam, rect);
  }
  // tiles the ellipse really meets inside its bounding rectangle, and the same by cells of 4 x 4 tiles: one
  // record (cell id, mask of the tiles met) per cell, which is what the binning sorts.
  unsigned int tiles = 0, nrec = 0;
  bool stored = false;
  {
    TileSpans sp;
    if (vis) sp.setup(g.u, g.v, g.A, g.B, g.C, g.tau, cam.W, cam.H);
    const int cx0 = rect[0] >> 2, cx1 = (rect[2] - 1) >> 2, cy0 = rect[1] >> 2, cy1 = (rect[3] - 1) >> 2;
    stored = vis && cx1 - cx0 <= 2 && cy1 - cy0 <= 2;          // at most 3 x 3 cells: the records fit the Gaussian's slots
    if (vis && !stored) {
      // a large footprint is only counted here (the record emission works its cells out again): a row of cells
      // contributes the cells from the leftmost to the rightmost tile met in its tile rows
      for (int cy = cy0; cy <= cy1; ++cy) {
        int lo = 1 << 30, hi = -1;
        const int ta = max(rect[1], 4 * cy), tb = min(rect[3], 4 * cy + 4);
        for (int ty = ta; ty < tb; ++ty) {
          int xa, xb;
          if (!sp.row(ty, rect[0], rect[2], xa, xb)) continue;
          tiles += (unsigned)(xb - xa);
          lo = min(lo, xa >> 2); hi = max(hi, (xb - 1) >> 2);
        }
        if (hi >= lo) nrec += (unsigned)(hi - lo + 1);
      }
    }
    // The tile rows of the other footprints are evaluated by the warp together, one (Gaussian, tile row) per lane
    // and round: lanes own very different numbers of rows (1 to 12), and a loop per lane would idle most of them.
    // Each owner parks its span parameters and the list of its rows in shared memory; a row's tiles go into the
    // owner's cell masks with shared-memory atomics (integer OR / add: any order gives the same bits).
    RowStage &rs = sRows[warp];
    const int rows = stored ? rect[3] - rect[1] : 0;
    int incl = rows;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const int t = __shfl_up_sync(kFull, incl, sft);
      if (lane >= sft) incl += t;
    }
    const int total = __shfl_sync(kFull, incl, 31);
    if (stored) {
      float *par = rs.par[lane];
      par[0] = sp.u; par[1] = sp.v; par[2] = sp.ila; par[3] = sp.lb; par[4] = sp.lc; par[5] = sp.taup; par[6] = sp.dys; par[7] = sp.eyp;
      rs.geo[lane] = make_int4(rect[0], rect[2], rect[1], cx0);
#pragma unroll
      for (int j = 0; j < 9; ++j) rs.mask[lane][j] = 0u;
      rs.tiles[lane] = 0u;
      for (int k = 0; k < rows; ++k) rs.list[incl - rows + k] = (unsigned short)((lane << 8) | k);
    }
    __syncwarp();
    for (int base = 0; base < total; base += 32) {
      if (base + lane < total) {
        const unsigned e = rs.list[base + lane];
        const int o = (int)(e >> 8), k = (int)(e & 255u);
        const float *par = rs.par[o];
        TileSpans so;
        so.u = par[0]; so.v = par[1]; so.ila = par[2]; so.lb = par[3]; so.lc = par[4]; so.taup = par[5]; so.dys = par[6]; so.eyp = par[7];
        so.W = cam.W; so.H = cam.H;
        const int4 ge = rs.geo[o];      // (tx0, tx1, ty0, first cell column)
        const int ty = ge.z + k;
        int xa, xb;
        if (so.row(ty, ge.x, ge.y, xa, xb)) {
          atomicAdd(&rs.tiles[o], (unsigned)(xb - xa));
          // the row's tiles as bits counted from the first column of the first cell (at most 12), a nibble per cell
          const uint32_t bits = ((1u << (xb - xa)) - 1u) << (xa - 4 * ge.w);
          const int cyi = (ty >> 2) - (ge.z >> 2), sh = 4 * (ty & 3);
#pragma unroll
          for (int c = 0; c < 3; ++c) {
            const uint32_t nib = (bits >> (4 * c)) & 15u;
            if (nib) atomicOr(&rs.mask[o][3 * cyi + c], nib << sh);
          }
        }
      }
    }
    __syncwarp();
    if (stored) {
      tiles = rs.tiles[lane];
      uint32_t *slot = a.cell_records + (size_t)i * kCellSlots;
#pragma unroll
      for (int j = 0; j < 9; ++j) {
        const uint32_t m = rs.mask[lane][j];
        if (m) slot[nrec++] = ((uint32_t)((cy0 + j / 3) * cam.cgx + cx0 + j % 3) << 16) | m;
      }
    }
    if (vis && tiles == 0) { vis = false; nrec = 0; rect[0] = rect[1] = rect[2] = rect[3] = 0; }
  }
  // ---- fused colour decode for the Gaussians that survived culling
  float pre[3] = {0.f, 0.f, 0.f};
  if (Explicit<APP>::value) {   // SH or Spherical Voronoi: parameter rows through the warp's slab
    float *slab = sData + warp * SlabOf<APP>::value;
    bool arrived = true;
    if (slab_by_copy) {
      __syncwarp();                         // lane 0 has initialised the barrier
      arrived = __all_sync(kFull, bulk::wait(bulk::smem_addr(sBar + warp), 0u));
      if (!arrived && lane == 0) atomicExch(a.pair_counter + 3, 1ull);   // reported by gs_async_status
    } else if (__any_sync(kFull, vis) && a.deg > 0 && row0 + 32 > a.n) {   // the ragged last warp
      warp_load_rows<RowOf<APP>::value>(a.sh_rest, row0, a.n, slab, lane);
    }
    if (vis && arrived) {
      float base[3];
      load3(a.base_color, i, base);
      SvCarry cy;
      explicit_pre<APP>(slab + lane * RowOf<APP>::value, base, g.dirx, g.diry, g.dirz, a.deg, pre, cy);
    }
  } else if (IsNeural<APP>::value) {
    float A[3] = {0.f, 0.f, 0.f};
    if (a.deg > 0 && __any_sync(kFull, vis)) {   // the whole warp decodes; culled lanes feed zeros
      float x[32];
      if (vis) {
        float f[8];
        load_features(a.features, i, f);
        decoder_inputs(g.dirx, g.diry, g.dirz, f, a.deg, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
      mlp::Activations act;
      // the lane's 14 words of the forward's weight operands come straight from global memory (1.6 KB that stay in L1)
      const mlp::FwdFrags F = mlp::load_fwd_frags(a.weights, lane);
      decode_warp<Split<APP>::value>(F, sStage[warp], lane, x, act, A);
    }
    if (vis) {
      float base[3];
      load3(a.base_color, i, base);
#pragma unroll
      for (int c = 0; c < 3; ++c) pre[c] = base[c] + 0.5f + A[c];
    }
  }
  if (in) {
    if (g.valid) {   // also for footprints that reach no tile: the tile stage is checked from these values
      reinterpret_cast<float2 *>(a.mean2d)[i] = make_float2(g.u, g.v);
      reinterpret_cast<float4 *>(a.conic_opacity)[i] = make_float4(g.A, g.B, g.C, g.o);
    }
    if (vis) {
      if (APP == kAppExternal) {   // the separate appearance pass reads the direction here and writes the colour over it
        a.color[3 * i] = g.dirx; a.color[3 * i + 1] = g.diry; a.color[3 * i + 2] = g.dirz;
      } else {
        a.color[3 * i] = color_act_z(a.act, pre[0]); a.color[3 * i + 1] = color_act_z(a.act, pre[1]); a.color[3 * i + 2] = color_act_z(a.act, pre[2]);
      }
    }
    a.depth_key[i] = vis ? g.zbits : 0xffffffffu;
    a.tiles_touched[i] = tiles;
    a.cell_count[i] = nrec | ((nrec && !stored) ? kCellBig : 0u);   // (vis was cleared if no tile is met: nrec = 0)
    reinterpret_cast<ushort4 *>(a.rect)[i] = make_ushort4((unsigned short)rect[0], (unsigned short)rect[1],
                                                          (unsigned short)rect[2], (unsigned short)rect[3]);
    if (a.extent) reinterpret_cast<float4 *>(a.extent)[i] = g.valid ? make_float4(g.ex, g.ey, g.tau, 0.f) : make_float4(-1.f, -1.f, 0.f, 0.f);
  }
  // ---- total number of (Gaussian, tile) instances
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) tiles += __shfl_xor_sync(kFull, tiles, s);
  if (lane == 0) sPairs[warp] = tiles;
  __syncthreads();
  if (tid == 0) {
    unsigned int tot = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) tot += sPairs[w];
    if (tot) atomicAdd(a.pair_counter, (unsigned long long)tot);
  }
}

// ---- backward of the projection for one Gaussian --------------------------------------------
struct GeoGrads { float mu[3], ls[3], q[4], logit; };

__device__ __forceinline__ GeoGrads project_backward(const float mu[3], const float ls[3], const float q[4],
                                                     float logit, const CamDev &cam, float gA, float gB,
                                                     float gC, float gu, float gv, float go, const float gd[3]) {
  GeoGrads out;
  // the same fast forms as the forward: gradients are held to 1e-3, these are good to a few ulp
  const float qi = rsqrtf(q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3]);
  const float r = q[0] * qi, x = q[1] * qi, y = q[2] * qi, z = q[3] * qi;
  float R[9];
  quat_rot(r, x, y, z, R);
  const float s[3] = {__expf(ls[0]), __expf(ls[1]), __expf(ls[2])};
  float M[9];
#pragma unroll
  for (int i = 0; i < 3; ++i)
#pragma unroll
    for (int k = 0; k < 3; ++k) M[3 * i + k] = R[3 * i + k] * s[k];
  const float tx = cam.R[0] * mu[0] + cam.R[1] * mu[1] + cam.R[2] * mu[2] + cam.t[0];
  const float ty = cam.R[3] * mu[0] + cam.R[4] * mu[1] + cam.R[5] * mu[2] + cam.t[1];
  const float tz = cam.R[6] * mu[0] + cam.R[7] * mu[1] + cam.R[8] * mu[2] + cam.t[2];
  const float iz = __fdividef(1.f, tz), iz2 = iz * iz;
  const float rx = tx * iz, ry = ty * iz;
  const bool clx = rx < -cam.limx || rx > cam.limx, cly = ry < -cam.limy || ry > cam.limy;
  const float txc = tz * fminf(cam.limx, fmaxf(-cam.limx, rx));
  const float tyc = tz * fminf(cam.limy, fmaxf(-cam.limy, ry));
  const float j00 = cam.fx * iz, j02 = -cam.fx * txc * iz2;
  const float j11 = cam.fy * iz, j12 = -cam.fy * tyc * iz2;
  float T[6];
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    T[c] = j00 * cam.R[c] + j02 * cam.R[6 + c];
    T[3 + c] = j11 * cam.R[3 + c] + j12 * cam.R[6 + c];
  }
  float N[6];  // N = T M, cov = N N^T + 0.3 I
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int c = 0; c < 3; ++c) N[3 * i + c] = T[3 * i] * M[c] + T[3 * i + 1] * M[3 + c] + T[3 * i + 2] * M[6 + c];
  const float a = N[0] * N[0] + N[1] * N[1] + N[2] * N[2] + kDilation;
  const float b = N[0] * N[3] + N[1] * N[4] + N[2] * N[5];
  const float c = N[3] * N[3] + N[4] * N[4] + N[5] * N[5] + kDilation;
  const float idet = __fdividef(1.f, cov_det(N, a, c));
  const float A = c * idet, B = -b * idet, C = a * idet;
  // conic -> covariance: G_cov = -Q G_Q Q, G_Q = [[gA, gB/2], [gB/2, gC]]
  const float h = 0.5f * gB;
  const float m00 = A * gA + B * h, m01 = A * h + B * gC, m10 = B * gA + C * h, m11 = B * h + C * gC;
  const float c00 = -(m00 * A + m01 * B), c01 = -(m00 * B + m01 * C), c11 = -(m10 * B + m11 * C);
  // cov = N N^T: G_N = 2 G_cov N (2x3); N = T M: G_T = G_N M^T, G_M = T^T G_N
  float GN[6];
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    GN[k] = 2.f * (c00 * N[k] + c01 * N[3 + k]);
    GN[3 + k] = 2.f * (c01 * N[k] + c11 * N[3 + k]);
  }
  float GT[6];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int k = 0; k < 3; ++k) GT[3 * i + k] = GN[3 * i] * M[3 * k] + GN[3 * i + 1] * M[3 * k + 1] + GN[3 * i + 2] * M[3 * k + 2];
  float GM[9];
#pragma unroll
  for (int i = 0; i < 3; ++i)
#pragma unroll
    for (int k = 0; k < 3; ++k) GM[3 * i + k] = T[i] * GN[k] + T[3 + i] * GN[3 + k];
  // T = J R_c: the four entries of G_J that exist
  const float gj00 = GT[0] * cam.R[0] + GT[1] * cam.R[1] + GT[2] * cam.R[2];
  const float gj02 = GT[0] * cam.R[6] + GT[1] * cam.R[7] + GT[2] * cam.R[8];
  const float gj11 = GT[3] * cam.R[3] + GT[4] * cam.R[4] + GT[5] * cam.R[5];
  const float gj12 = GT[3] * cam.R[6] + GT[4] * cam.R[7] + GT[5] * cam.R[8];
  float gtx = gu * cam.fx * iz, gty = gv * cam.fy * iz;
  float gtz = -(gu * cam.fx * tx + gv * cam.fy * ty) * iz2 - (gj00 * cam.fx + gj11 * cam.fy) * iz2;
  if (!clx) { gtx -= gj02 * cam.fx * iz2; gtz += gj02 * 2.f * cam.fx * tx * iz2 * iz; }
  else      { gtz -= gj02 * j02 * iz; }
  if (!cly) { gty -= gj12 * cam.fy * iz2; gtz += gj12 * 2.f * cam.fy * ty * iz2 * iz; }
  else      { gtz -= gj12 * j12 * iz; }
  // direction d = (mu - o_c)/|mu - o_c|: tangent projection of dL/dd
  const float vx = mu[0] - cam.oc[0], vy = mu[1] - cam.oc[1], vz = mu[2] - cam.oc[2];
  const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
  const float dx = vx * vi, dy = vy * vi, dz = vz * vi;
  const float dot = dx * gd[0] + dy * gd[1] + dz * gd[2];
  out.mu[0] = cam.R[0] * gtx + cam.R[3] * gty + cam.R[6] * gtz + (gd[0] - dx * dot) * vi;
  out.mu[1] = cam.R[1] * gtx + cam.R[4] * gty + cam.R[7] * gtz + (gd[1] - dy * dot) * vi;
  out.mu[2] = cam.R[2] * gtx + cam.R[5] * gty + cam.R[8] * gtz + (gd[2] - dz * dot) * vi;
  // M = R diag(s)
  float D[9];
#pragma unroll
  for (int k = 0; k < 3; ++k) {
    const float gs = GM[k] * R[k] + GM[3 + k] * R[3 + k] + GM[6 + k] * R[6 + k];
    out.ls[k] = s[k] * gs;
    D[k] = GM[k] * s[k]; D[3 + k] = GM[3 + k] * s[k]; D[6 + k] = GM[6 + k] * s[k];
  }
  float gq[4];
  gq[0] = 2.f * (z * (D[3] - D[1]) + y * (D[2] - D[6]) + x * (D[7] - D[5]));
  gq[1] = 2.f * (y * (D[1] + D[3]) + z * (D[2] + D[6]) + r * (D[7] - D[5]) - 2.f * x * (D[4] + D[8]));
  gq[2] = 2.f * (x * (D[1] + D[3]) + r * (D[2] - D[6]) + z * (D[5] + D[7]) - 2.f * y * (D[0] + D[8]));
  gq[3] = 2.f * (r * (D[3] - D[1]) + x * (D[2] + D[6]) + y * (D[5] + D[7]) - 2.f * z * (D[0] + D[4]));
  const float qd = r * gq[0] + x * gq[1] + y * gq[2] + z * gq[3];
  out.q[0] = (gq[0] - r * qd) * qi; out.q[1] = (gq[1] - x * qd) * qi;
  out.q[2] = (gq[2] - y * qd) * qi; out.q[3] = (gq[3] - z * qd) * qi;
  const float o = __fdividef(1.f, 1.f + __expf(-logit));
  out.logit = go * o * (1.f - o);
  return out;
}

__device__ __forceinline__ void store3(float *p, int64_t i, float a, float b, float c) {
  p[3 * i] = a; p[3 * i + 1] = b; p[3 * i + 2] = c;
}

// Shared memory of the backward kernels (dynamic): SH: kWarps slabs of coefficient rows.
// Neural: weights [816] | kWarps operand slabs [32][100] (reused as [kWarps][816] at the end).
constexpr size_t kBwdSmemSH = sizeof(float) * kWarps * SlabOf<GS_APP_SH>::value;
constexpr size_t kBwdSmemSV = sizeof(float) * kWarps * SlabOf<GS_APP_SV>::value;
constexpr size_t kBwdSmemNN = sizeof(mlp::Weights) + kWarps * sizeof(mlp::WarpStage);
static_assert(kWarps * sizeof(mlp::WarpStage) >= kWarps * GS_MLP_WEIGHTS * sizeof(float), "partial sums reuse the staging areas");
static_assert(sizeof(mlp::Weights) % 16 == 0, "staging areas must stay 16-byte aligned");

template <int APP>
__global__ void __launch_bounds__(kBlock) k_preprocess_bwd(PreprocessBwdArgs a, CamDev cam) {
  dependency_wait();
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float *slab = smem + warp * SlabOf<APP>::value;   // SH / SV: this warp's slab of parameter rows
  mlp::Weights &sWt = *reinterpret_cast<mlp::Weights *>(smem);
  mlp::WarpStage *sStage = reinterpret_cast<mlp::WarpStage *>(reinterpret_cast<unsigned char *>(smem) + sizeof(mlp::Weights));
  mlp::WeightGrad dW;
  if (IsNeural<APP>::value) {
    mlp::load_weights(a.weights, sWt, tid, kBlock);
    dW.clear();
    __syncthreads();
  }
  // SH / Spherical Voronoi: the warp's slab of parameter rows comes in by one bulk copy and its slab of gradient
  // rows leaves by one (a ragged last warp uses plain loads and stores)
  __shared__ unsigned long long sBar[kWarps];
  uint32_t slab_parity = 0u;
  if (Explicit<APP>::value && lane == 0) {
    bulk::barrier_init(bulk::smem_addr(sBar + warp));
    bulk::fence_barrier_init();
  }
  __syncwarp();
  const int64_t nchunks = (a.n + kBlock - 1) / kBlock;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    reload_fence();
    const int64_t i = chunk * kBlock + tid;
    const int64_t row0 = chunk * kBlock + warp * 32;
    const bool in = i < a.n;
    // Every input row of this Gaussian is requested here, before anything depends on one of them (also for
    // culled Gaussians, whose rows are then ignored): one memory round trip per trip of the loop instead of one
    // per branch that needs a value.
    bool vis = false;
    float gd[3] = {0.f, 0.f, 0.f};
    float mu[3] = {0.f, 0.f, 0.f}, ls[3] = {0.f, 0.f, 0.f}, q[4] = {1.f, 0.f, 0.f, 0.f}, logit = 0.f;
    float4 ga = make_float4(0.f, 0.f, 0.f, 0.f), gb = ga, gc = ga;
    float base_in[3] = {0.f, 0.f, 0.f};
    uint4 feat_raw = make_uint4(0u, 0u, 0u, 0u);
    float dx = 0.f, dy = 0.f, dz = 0.f;
    if (in) {
      const ushort4 rc = __ldg(reinterpret_cast<const ushort4 *>(a.rect) + i);
      load3(a.means, i, mu);
      load3(a.log_scales, i, ls);
      const float4 q4 = __ldg(reinterpret_cast<const float4 *>(a.quats) + i);
      logit = __ldg(a.logits + i);
      const float4 *g2 = reinterpret_cast<const float4 *>(a.g2d) + 3 * i;
      ga = g2[0]; gb = g2[1]; gc = g2[2];   // (gr, gg, gb, go) (gA, gB, gC, gu) (gv, -, -, -)
      if (APP != kAppExternal) load3(a.base_color, i, base_in);
      else load3(a.gd_in, i, gd);
      if (IsNeural<APP>::value) feat_raw = __ldg(reinterpret_cast<const uint4 *>(a.features) + i);
      q[0] = q4.x; q[1] = q4.y; q[2] = q4.z; q[3] = q4.w;
      vis = rc.z > rc.x && rc.w > rc.y;
    }
    const bool warp_vis = __any_sync(kFull, vis);
    const bool full_warp = row0 + 32 <= a.n;
    const bool slab_by_copy = Explicit<APP>::value && warp_vis && a.deg > 0 && full_warp;
    if (Explicit<APP>::value && lane == 0) {
      bulk::wait_stores_read();          // an earlier trip's gradient slab has left shared memory
      if (slab_by_copy)
        bulk::load(bulk::smem_addr(slab), a.sh_rest + row0 * RowOf<APP>::value, SlabOf<APP>::value * sizeof(float),
                   bulk::smem_addr(sBar + warp));
    }
    if (Explicit<APP>::value) __syncwarp();
    if (vis) {
      const float vx = mu[0] - cam.oc[0], vy = mu[1] - cam.oc[1], vz = mu[2] - cam.oc[2];
      const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
      dx = vx * vi; dy = vy * vi; dz = vz * vi;
    }
    // ---- appearance backward
    float gp[3] = {0.f, 0.f, 0.f};
    if (APP == kAppExternal) {
      // dL/dd came from the separate appearance backward (zero rows for culled Gaussians)
    } else if (Explicit<APP>::value) {
      if (row0 < a.n) {
        bool arrived = true;
        if (slab_by_copy) {
          arrived = __all_sync(kFull, bulk::wait(bulk::smem_addr(sBar + warp), slab_parity));
          slab_parity ^= 1u;
          if (!arrived && lane == 0 && a.timeout) atomicExch(a.timeout, 1ull);   // reported by gs_async_status
        } else if (warp_vis && a.deg > 0) {
          warp_load_rows<RowOf<APP>::value>(a.sh_rest, row0, a.n, slab, lane);
        }
        float *row = slab + lane * RowOf<APP>::value;
        if (vis && arrived) {
          float pre[3];
          const float (&base)[3] = base_in;
          SvCarry cy;
          if (a.deg > 0) explicit_pre<APP>(row, base, dx, dy, dz, a.deg, pre, cy);
          else { pre[0] = base[0] + 0.5f; pre[1] = base[1] + 0.5f; pre[2] = base[2] + 0.5f; }
          gp[0] = color_act_grad_z(a.act, pre[0]) * ga.x; gp[1] = color_act_grad_z(a.act, pre[1]) * ga.y;
          gp[2] = color_act_grad_z(a.act, pre[2]) * ga.z;
          explicit_bwd<APP>(row, gp, dx, dy, dz, a.deg, cy, gd);
        } else {
#pragma unroll
          for (int k = 0; k < RowOf<APP>::value; ++k) row[k] = 0.f;
        }
        if (full_warp) {
          bulk::fence_generic_writes();     // the lanes' rows become visible to the copy engine
          __syncwarp();
          if (lane == 0) bulk::store(a.g_sh_rest + row0 * RowOf<APP>::value, bulk::smem_addr(slab), SlabOf<APP>::value * sizeof(float));
        } else {
          warp_store_rows<RowOf<APP>::value>(a.g_sh_rest, row0, a.n, slab, lane);
        }
      }
    } else {
      float gf[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      float base[3] = {0.f, 0.f, 0.f};
      const float gcol[3] = {ga.x, ga.y, ga.z};
      if (vis) { base[0] = base_in[0]; base[1] = base_in[1]; base[2] = base_in[2]; }
      if (warp_vis && a.deg > 0) {   // the whole warp goes through the decoder; culled lanes feed zeros
        float x[32];
        if (vis) {
          float f[8];
          unpack_features(feat_raw, f);
          decoder_inputs(dx, dy, dz, f, a.deg, x);
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) x[k] = 0.f;
        }
        decode_backward_warp<Split<APP>::value>(sWt, sStage[warp], lane, vis, x, dx, dy, dz, a.deg, a.act, base, gcol, dW, gp, gf, gd);
      } else if (vis) {
#pragma unroll
        for (int c = 0; c < 3; ++c) gp[c] = color_act_grad_z(a.act, base[c] + 0.5f) * gcol[c];
      }
      if (in) {
        float4 *gfp = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
        gfp[0] = make_float4(gf[0], gf[1], gf[2], gf[3]);
        gfp[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      }
    }
    // ---- geometry backward
    if (in) {
      GeoGrads gg;
      if (vis) {
        gg = project_backward(mu, ls, q, logit, cam, gb.x, gb.y, gb.z, gb.w, gc.x, ga.w, gd);
      } else {
#pragma unroll
        for (int k = 0; k < 3; ++k) { gg.mu[k] = 0.f; gg.ls[k] = 0.f; }
#pragma unroll
        for (int k = 0; k < 4; ++k) gg.q[k] = 0.f;
        gg.logit = 0.f;
      }
      store3(a.g_means, i, gg.mu[0], gg.mu[1], gg.mu[2]);
      store3(a.g_log_scales, i, gg.ls[0], gg.ls[1], gg.ls[2]);
      reinterpret_cast<float4 *>(a.g_quats)[i] = make_float4(gg.q[0], gg.q[1], gg.q[2], gg.q[3]);
      a.g_logits[i] = gg.logit;
      if (APP != kAppExternal) store3(a.g_base, i, gp[0], gp[1], gp[2]);
    }
  }
  if (IsNeural<APP>::value) {
    weight_grad_flush(dW, reinterpret_cast<float *>(sStage), a.w_partials + (size_t)blockIdx.x * GS_MLP_WEIGHTS, tid);
  }
  if (Explicit<APP>::value && lane == 0) bulk::wait_stores_done();
}

// ---- preprocess backward over the Gaussians that received a gradient -------------------------------------------
// A Gaussian whose nine 2D gradients are all zero - culled, or listed in tiles but composited by no pixel of this view
// because the pixels it covers saturated in front of it - gets zero gradients whatever its parameters are.  In a
// scene with occlusion that is most of them (config 3: 94 % of the visible Gaussians of a view).  Two kernels:
// k_bwd_flags streams over all Gaussians at full occupancy, writes the zero rows and leaves one bit per Gaussian
// (set = it received a gradient); k_preprocess_bwd_sparse, persistent, gathers the flagged ones in index order and,
// whenever kBlock of them are queued, runs them through the decoder and projection backward, one per thread, with
// every lane busy.  A CTA's run of flag words is fixed by the grid, so the order of all sums is the same from run to
// run.
constexpr int kFlagThreads = 256;
template <bool kBase, bool kFeatures>
__global__ void __launch_bounds__(kFlagThreads) k_bwd_flags(PreprocessBwdArgs a) {
  dependency_wait();
  const int64_t i = (int64_t)blockIdx.x * kFlagThreads + threadIdx.x;
  bool active = false;
  if (i < a.n) {
    const ushort4 rc = __ldg(reinterpret_cast<const ushort4 *>(a.rect) + i);
    if (rc.z > rc.x && rc.w > rc.y) {
      const float4 *g2 = reinterpret_cast<const float4 *>(a.g2d) + 3 * i;
      const float4 ga = g2[0], gb = g2[1];
      const float gv = a.g2d[12 * i + 8];
      active = ga.x != 0.f || ga.y != 0.f || ga.z != 0.f || ga.w != 0.f || gb.x != 0.f || gb.y != 0.f || gb.z != 0.f ||
               gb.w != 0.f || gv != 0.f;
    }
    if (!active) {
      store3(a.g_means, i, 0.f, 0.f, 0.f);
      store3(a.g_log_scales, i, 0.f, 0.f, 0.f);
      reinterpret_cast<float4 *>(a.g_quats)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      a.g_logits[i] = 0.f;
      if (kBase) store3(a.g_base, i, 0.f, 0.f, 0.f);
      if (kFeatures) {
        const int quads = a.nfeat == 16 ? 4 : 2;
        float4 *gfp = reinterpret_cast<float4 *>(a.g_features) + quads * i;
        for (int q = 0; q < quads; ++q) gfp[q] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
  const unsigned ballot = __ballot_sync(kFull, active);
  if ((threadIdx.x & 31) == 0 && i < a.n) a.flags[i >> 5] = ballot;    // (i is a multiple of 32 here)
}

template <int APP>
__global__ void __launch_bounds__(kBlock) k_preprocess_bwd_sparse(PreprocessBwdArgs a, CamDev cam) {
  dependency_wait();
  static_assert(IsNeural<APP>::value || APP == kAppExternal, "the neural model, or the projection alone");
  extern __shared__ __align__(16) float smem[];
  constexpr int kWordsPerRound = kBlock / 4;             // flag words (of 32 Gaussians) looked at per round
  __shared__ uint32_t s_queue[2 * 32 * kWordsPerRound];  // a power of two above 32 * kWordsPerRound + kBlock - 1
  __shared__ int s_warp_count[kWarps];
  constexpr int kMask = 2 * 32 * kWordsPerRound - 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  mlp::Weights &sWt = *reinterpret_cast<mlp::Weights *>(smem);
  mlp::WarpStage *sStage = reinterpret_cast<mlp::WarpStage *>(reinterpret_cast<unsigned char *>(smem) + sizeof(mlp::Weights));
  mlp::WeightGrad dW;
  if (IsNeural<APP>::value) {
    mlp::load_weights(a.weights, sWt, tid, kBlock);
    dW.clear();
    __syncthreads();
  }
  int q_head = 0, q_count = 0;      // the same in every thread

  // the first `count` queued Gaussians, one per thread
  auto process = [&](int count) {
    const bool has = tid < count;
    const int64_t i = has ? (int64_t)s_queue[(q_head + tid) & kMask] : 0;
    float gd[3] = {0.f, 0.f, 0.f};
    float mu[3] = {0.f, 0.f, 0.f}, ls[3] = {0.f, 0.f, 0.f}, q[4] = {1.f, 0.f, 0.f, 0.f}, logit = 0.f;
    float4 ga = make_float4(0.f, 0.f, 0.f, 0.f), gb = ga, gc = ga;
    float base[3] = {0.f, 0.f, 0.f};
    uint4 feat_raw = make_uint4(0u, 0u, 0u, 0u);
    float dx = 0.f, dy = 0.f, dz = 1.f;
    if (has) {
      load3(a.means, i, mu);
      load3(a.log_scales, i, ls);
      const float4 q4 = __ldg(reinterpret_cast<const float4 *>(a.quats) + i);
      logit = __ldg(a.logits + i);
      const float4 *g2 = reinterpret_cast<const float4 *>(a.g2d) + 3 * i;
      ga = g2[0]; gb = g2[1]; gc = g2[2];
      if (APP != kAppExternal) load3(a.base_color, i, base);
      else load3(a.gd_in, i, gd);
      if (IsNeural<APP>::value) feat_raw = __ldg(reinterpret_cast<const uint4 *>(a.features) + i);
      q[0] = q4.x; q[1] = q4.y; q[2] = q4.z; q[3] = q4.w;
      const float vx = mu[0] - cam.oc[0], vy = mu[1] - cam.oc[1], vz = mu[2] - cam.oc[2];
      const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
      dx = vx * vi; dy = vy * vi; dz = vz * vi;
    }
    float gp[3] = {0.f, 0.f, 0.f};
    if (IsNeural<APP>::value) {
      float gf[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      const float gcol[3] = {ga.x, ga.y, ga.z};
      if (warp * 32 < count && a.deg > 0) {     // the whole warp goes through the decoder; lanes past the count feed zeros
        float x[32];
        if (has) {
          float f[8];
          unpack_features(feat_raw, f);
          decoder_inputs(dx, dy, dz, f, a.deg, x);
        } else {
#pragma unroll
          for (int k = 0; k < 32; ++k) x[k] = 0.f;
        }
        decode_backward_warp<Split<APP>::value>(sWt, sStage[warp], lane, has, x, dx, dy, dz, a.deg, a.act, base, gcol, dW, gp, gf, gd);
      } else if (has) {
#pragma unroll
        for (int c = 0; c < 3; ++c) gp[c] = color_act_grad_z(a.act, base[c] + 0.5f) * gcol[c];
      }
      if (has) {
        float4 *gfp = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
        gfp[0] = make_float4(gf[0], gf[1], gf[2], gf[3]);
        gfp[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      }
    }
    if (has) {
      const GeoGrads gg = project_backward(mu, ls, q, logit, cam, gb.x, gb.y, gb.z, gb.w, gc.x, ga.w, gd);
      store3(a.g_means, i, gg.mu[0], gg.mu[1], gg.mu[2]);
      store3(a.g_log_scales, i, gg.ls[0], gg.ls[1], gg.ls[2]);
      reinterpret_cast<float4 *>(a.g_quats)[i] = make_float4(gg.q[0], gg.q[1], gg.q[2], gg.q[3]);
      a.g_logits[i] = gg.logit;
      if (APP != kAppExternal) store3(a.g_base, i, gp[0], gp[1], gp[2]);
    }
  };

  // The flags of k_bwd_flags, one bit per Gaussian, say who is left.  Every CTA takes one contiguous run of flag words
  // (equal to within a word whatever the grid) and reads it kWordsPerRound words at a time: thread t looks at byte
  // t % 4 of word t / 4, an exclusive scan over the CTA gives its place in the queue, and it writes the indices of its
  // set bits there - index order, the same from run to run.
  const int64_t nwords = (a.n + 31) / 32, per_cta = (nwords + gridDim.x - 1) / gridDim.x;
  const int64_t w_begin = min(nwords, (int64_t)blockIdx.x * per_cta), w_end = min(nwords, w_begin + per_cta);
  for (int64_t w0 = w_begin; w0 < w_end; w0 += kWordsPerRound) {
    reload_fence();
    const int64_t w = w0 + (tid >> 2);
    const uint32_t byte = w < w_end ? (__ldg(a.flags + w) >> (8 * (tid & 3))) & 255u : 0u;
    const int cnt = __popc(byte);
    int incl = cnt;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const int t = __shfl_up_sync(kFull, incl, sft);
      if (lane >= sft) incl += t;
    }
    if (lane == 31) s_warp_count[warp] = incl;
    __syncthreads();
    int offset = incl - cnt, total = 0;
#pragma unroll
    for (int ww = 0; ww < kWarps; ++ww) { const int c = s_warp_count[ww]; offset += ww < warp ? c : 0; total += c; }
    uint32_t bits = byte;
    const uint32_t row0 = (uint32_t)(w * 32 + 8 * (tid & 3));
    for (int slot = q_head + q_count + offset; bits; ++slot) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1u;
      s_queue[slot & kMask] = row0 + (uint32_t)b;
    }
    __syncthreads();
    q_count += total;
    while (q_count >= kBlock) {
      process(kBlock);
      q_head = (q_head + kBlock) & kMask;
      q_count -= kBlock;
      __syncthreads();
    }
  }
  if (q_count > 0) process(q_count);
  if (IsNeural<APP>::value) {
    weight_grad_flush(dW, reinterpret_cast<float *>(sStage), a.w_partials + (size_t)blockIdx.x * GS_MLP_WEIGHTS, tid);
  }
}

// ---- separate-pass appearance kernels of the neural model (the explicit models follow, with bulk copies) ------
#include "gs_decoder_tc.cuh"

template <int APP>
__global__ void __launch_bounds__(kBlock) k_appearance_fwd(AppearanceArgs a) {
  static_assert(IsNeural<APP>::value, "the neural model in either decoder precision");
  __shared__ __align__(16) StageFwd sStage[kWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // persistent: the forward's weight operands are read once into 14 registers per lane and serve every trip
  const mlp::FwdFrags F = mlp::load_fwd_frags(a.weights, lane);
  const int64_t nchunks = (a.n + kBlock - 1) / kBlock;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int64_t i = chunk * kBlock + tid;
    const int64_t row0 = chunk * kBlock + warp * 32;
    const bool in = i < a.n && (!a.mask || __ldg(a.mask + i) != 0u);   // masked-out Gaussians are skipped
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, A[3] = {0.f, 0.f, 0.f};
    if (in) { load3(a.dirs, i, d); load3(a.base_color, i, base); }
    if (a.deg > 0 && row0 < a.n) {   // the whole warp decodes; lanes without a Gaussian feed zeros
      float x[32];
      if (in) {
        float f[8];
        load_features(a.features, i, f);
        decoder_inputs(d[0], d[1], d[2], f, a.deg, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
      mlp::Activations act;
      decode_warp<Split<APP>::value>(F, sStage[warp], lane, x, act, A);
      __syncwarp();   // the staging area is free for the next trip
    }
    if (in)
      store3(a.color, i, color_act_z(a.act, base[0] + 0.5f + A[0]), color_act_z(a.act, base[1] + 0.5f + A[1]),
             color_act_z(a.act, base[2] + 0.5f + A[2]));
  }
}

template <int APP>
__global__ void __launch_bounds__(kBlock) k_appearance_bwd(AppearanceArgs a) {
  static_assert(IsNeural<APP>::value, "the neural model in either decoder precision");
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  mlp::Weights &sWt = *reinterpret_cast<mlp::Weights *>(smem);
  mlp::WarpStage *sStage = reinterpret_cast<mlp::WarpStage *>(reinterpret_cast<unsigned char *>(smem) + sizeof(mlp::Weights));
  mlp::WeightGrad dW;
  mlp::load_weights(a.weights, sWt, tid, kBlock);
  dW.clear();
  __syncthreads();
  const int64_t nchunks = (a.n + kBlock - 1) / kBlock;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    reload_fence();
    const int64_t i = chunk * kBlock + tid;
    const int64_t row0 = chunk * kBlock + warp * 32;
    const bool exists = i < a.n;
    const bool in = exists && (!a.mask || __ldg(a.mask + i) != 0u);   // masked out: zero gradient rows
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, gcol[3] = {0.f, 0.f, 0.f};
    if (in) { load3(a.dirs, i, d); load3(a.base_color, i, base); load3(a.g_color, i, gcol); }
    float gp[3] = {0.f, 0.f, 0.f}, gd[3] = {0.f, 0.f, 0.f};
    float gf[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (a.deg > 0 && row0 < a.n) {
      float x[32];
      if (in) {
        float f[8];
        load_features(a.features, i, f);
        decoder_inputs(d[0], d[1], d[2], f, a.deg, x);
      } else {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = 0.f;
      }
      decode_backward_warp<Split<APP>::value>(sWt, sStage[warp], lane, in, x, d[0], d[1], d[2], a.deg, a.act, base, gcol, dW, gp, gf, gd);
    } else if (in) {
#pragma unroll
      for (int c = 0; c < 3; ++c) gp[c] = color_act_grad_z(a.act, base[c] + 0.5f) * gcol[c];
    }
    if (exists) {
      float4 *gfp = reinterpret_cast<float4 *>(a.g_features) + 2 * i;
      gfp[0] = make_float4(gf[0], gf[1], gf[2], gf[3]);
      gfp[1] = make_float4(gf[4], gf[5], gf[6], gf[7]);
      store3(a.g_base, i, gp[0], gp[1], gp[2]);
      store3(a.g_dirs, i, gd[0], gd[1], gd[2]);
    }
  }
  weight_grad_flush(dW, reinterpret_cast<float *>(sStage), a.w_partials + (size_t)blockIdx.x * GS_MLP_WEIGHTS, tid);
}

// ---- separate-pass kernels of the explicit models with bulk copies ---------------------------------------------
// The parameter rows of a warp's 32 Gaussians are one contiguous piece of global memory (5760 B for SH, 6272 B
// for Spherical Voronoi, a multiple of 16 either way).  One lane moves it with a single 1D bulk copy of the
// tensor memory accelerator into the warp's shared-memory slab and the warp sleeps on an mbarrier until the
// bytes have landed; the gradient slab of the backward goes back the same way.  Each warp owns two slabs and is
// persistent, so the copy of its next 32 rows is in flight while it works on the current ones, with no
// registers or store instructions spent on staging.  Every wait is bounded: if a barrier does not flip within
// the limit the warp records it in *timeout and leaves, draining its own copies first.

template <int APP> constexpr size_t bulk_smem_bytes() {
  return sizeof(float) * kWarps * 2 * SlabOf<APP>::value + sizeof(unsigned long long) * kWarps * 2;
}

// BWD = false: colours.  BWD = true: gradient rows (written in place over the parameter rows), dL/dc0, dL/dd.
template <int APP, bool BWD>
__global__ void __launch_bounds__(kBlock) k_appearance_bulk(AppearanceArgs a) {
  static_assert(Explicit<APP>::value, "the explicit models only");
  constexpr int kRow = RowOf<APP>::value, kSlab = SlabOf<APP>::value;
  constexpr uint32_t kBytes = kSlab * sizeof(float);
  static_assert(kBytes % 16 == 0, "a bulk copy moves multiples of 16 bytes");
  extern __shared__ __align__(128) unsigned char bulk_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float *const buf0 = reinterpret_cast<float *>(bulk_smem) + (warp * 2) * kSlab, *const buf1 = buf0 + kSlab;
  unsigned long long *bars = reinterpret_cast<unsigned long long *>(bulk_smem + sizeof(float) * kWarps * 2 * kSlab);
  const uint32_t bar0 = bulk::smem_addr(bars + warp * 2), bar1 = bar0 + 8;
  if (lane == 0) {
    bulk::barrier_init(bar0); bulk::barrier_init(bar1);
    bulk::fence_barrier_init();
  }
  __syncwarp();
  const bool rows_needed = a.deg > 0;
  const int64_t nchunks = (a.n + kBlock - 1) / kBlock;
  uint32_t parity0 = 0u, parity1 = 0u;   // phase each barrier completes next
  int s = 0;
  // the first copy
  {
    const int64_t row0 = (int64_t)blockIdx.x * kBlock + warp * 32;
    if (rows_needed && lane == 0 && row0 + 32 <= a.n) bulk::load(bulk::smem_addr(buf0), a.sh_rest + row0 * kRow, kBytes, bar0);
  }
  bool ok = true;
  for (int64_t chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x, s ^= 1) {
    const int64_t row0 = chunk * kBlock + warp * 32, i = row0 + lane;
    const int rows = row0 < a.n ? (int)min((int64_t)32, a.n - row0) : 0;
    __syncwarp();                      // every lane is done with the other slab
    if (lane == 0) {
      if (BWD) bulk::wait_stores_read();   // ... and so is the copy that carried its gradients away
      const int64_t nrow0 = row0 + (int64_t)gridDim.x * kBlock;
      if (rows_needed && nrow0 + 32 <= a.n) bulk::load(bulk::smem_addr(s ? buf0 : buf1), a.sh_rest + nrow0 * kRow, kBytes, s ? bar0 : bar1);
    }
    if (rows == 0) continue;
    const bool exists = lane < rows;
    const bool in = exists && (!a.mask || __ldg(a.mask + i) != 0u);
    float d[3] = {0.f, 0.f, 1.f}, base[3] = {0.f, 0.f, 0.f}, gcol[3] = {0.f, 0.f, 0.f};
    if (in) {
      load3(a.dirs, i, d); load3(a.base_color, i, base);
      if (BWD) load3(a.g_color, i, gcol);
    }
    float *slab = s ? buf1 : buf0, *row = slab + lane * kRow;
    if (rows_needed) {
      if (rows == 32) {
        ok = bulk::wait(s ? bar1 : bar0, s ? parity1 : parity0);
        if (s) parity1 ^= 1u; else parity0 ^= 1u;
        if (!__all_sync(kFull, ok)) { ok = false; break; }
      } else {
        __syncwarp();
        warp_load_rows<kRow>(a.sh_rest, row0, a.n, slab, lane);   // the ragged last rows: plain loads
      }
    }
    float pre[3] = {base[0] + 0.5f, base[1] + 0.5f, base[2] + 0.5f};
    SvCarry cy;
    if (in && rows_needed) explicit_pre<APP>(row, base, d[0], d[1], d[2], a.deg, pre, cy);
    if (!BWD) {
      if (in) store3(a.color, i, color_act_z(a.act, pre[0]), color_act_z(a.act, pre[1]), color_act_z(a.act, pre[2]));
    } else {
      float gp[3] = {0.f, 0.f, 0.f}, gd[3] = {0.f, 0.f, 0.f};
      if (in) {
#pragma unroll
        for (int c = 0; c < 3; ++c) gp[c] = color_act_grad_z(a.act, pre[c]) * gcol[c];
        explicit_bwd<APP>(row, gp, d[0], d[1], d[2], a.deg, cy, gd);
      } else if (exists) {
#pragma unroll
        for (int k = 0; k < kRow; ++k) row[k] = 0.f;
      }
      if (exists) {
        store3(a.g_base, i, gp[0], gp[1], gp[2]);
        store3(a.g_dirs, i, gd[0], gd[1], gd[2]);
      }
      if (rows == 32) {
        bulk::fence_generic_writes();      // the lanes' rows become visible to the copy engine
        __syncwarp();
        if (lane == 0) bulk::store(a.g_sh_rest + row0 * kRow, bulk::smem_addr(slab), kBytes);
      } else {
        warp_store_rows<kRow>(a.g_sh_rest, row0, a.n, slab, lane);
      }
    }
  }
  if (lane == 0) {
    if (BWD) bulk::wait_stores_done();
    if (!ok && a.timeout) atomicExch(a.timeout, 1ull);
  }
  if (!ok && rows_needed) {
    // a copy may still be in flight into this warp's slabs: give it the same bounded time before the CTA ends
    bulk::wait(bar0, parity0);
    bulk::wait(bar1, parity1);
  }
}

// Unfused step, backward: what the separate appearance backward reads, as dense arrays.
__global__ void __launch_bounds__(kBlock) k_unfused_prepare(int64_t n, const float *__restrict__ means, CamDev cam,
                                                            const float *__restrict__ g2d, const uint32_t *__restrict__ mask,
                                                            float *__restrict__ dirs, float *__restrict__ g_color) {
  const int64_t i = (int64_t)blockIdx.x * kBlock + threadIdx.x;
  if (i >= n) return;
  float d[3] = {0.f, 0.f, 1.f}, g[3] = {0.f, 0.f, 0.f};
  if (__ldg(mask + i) != 0u) {
    float mu[3];
    load3(means, i, mu);
    const float vx = mu[0] - cam.oc[0], vy = mu[1] - cam.oc[1], vz = mu[2] - cam.oc[2];
    const float vi = rsqrtf(vx * vx + vy * vy + vz * vz);
    d[0] = vx * vi; d[1] = vy * vi; d[2] = vz * vi;
    const float4 ga = __ldg(reinterpret_cast<const float4 *>(g2d) + 3 * i);
    g[0] = ga.x; g[1] = ga.y; g[2] = ga.z;
  }
  store3(dirs, i, d[0], d[1], d[2]);
  store3(g_color, i, g[0], g[1], g[2]);
}

inline int grid_for(int64_t n) { return (int)((n + kBlock - 1) / kBlock); }

template <class K>
void opt_in_smem(K kernel, size_t bytes) {
  cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Grid of a persistent kernel: as many CTAs as fit on the device at once (a second, thinner wave of a
// grid-stride loop would run at a fraction of the occupancy), at most kWgradBlocks (rows of the partial buffer).
template <auto kernel>      // one cache per kernel, not per signature
int resident_blocks(size_t smem_bytes, int cap = kWgradBlocks) {
  static int cached[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) return kWgradBlocks;
  if (!cached[dev]) {
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kBlock, smem_bytes) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || per_sm <= 0 || sms <= 0)
      return kWgradBlocks;
    cached[dev] = per_sm * sms < cap ? per_sm * sms : cap;
  }
  return cached[dev];
}

}  // namespace

int launch_preprocess_fwd(int app, const PreprocessArgs &a, const CamDev &cam, cudaStream_t st) {
  if (a.n == 0) return 0;
  if (app == GS_APP_SH) launch_chained(k_preprocess_fwd<GS_APP_SH>, grid_for(a.n), kBlock, 0, st, a, cam);
  else if (app == GS_APP_SV) launch_chained(k_preprocess_fwd<GS_APP_SV>, grid_for(a.n), kBlock, 0, st, a, cam);
  else if (app == kAppExternal) launch_chained(k_preprocess_fwd<kAppExternal>, grid_for(a.n), kBlock, 0, st, a, cam);
  else if (app == kAppNeuralHalf) launch_chained(k_preprocess_fwd<kAppNeuralHalf>, grid_for(a.n), kBlock, 0, st, a, cam);
  else launch_chained(k_preprocess_fwd<GS_APP_NEURAL>, grid_for(a.n), kBlock, 0, st, a, cam);
  return 1;
}

int launch_unfused_prepare(int64_t n, const float *means, const CamDev &cam, const float *g2d, const uint32_t *mask,
                           float *dirs, float *g_color, cudaStream_t st) {
  if (n == 0) return 0;
  k_unfused_prepare<<<grid_for(n), kBlock, 0, st>>>(n, means, cam, g2d, mask, dirs, g_color);
  return 1;
}

int launch_bwd_flags(const PreprocessBwdArgs &a, bool appearance_rows, cudaStream_t st) {
  if (a.n == 0) return 0;
  const int blocks = (int)((a.n + kFlagThreads - 1) / kFlagThreads);
  if (appearance_rows) launch_chained(k_bwd_flags<true, true>, blocks, kFlagThreads, 0, st, a);
  else launch_chained(k_bwd_flags<false, false>, blocks, kFlagThreads, 0, st, a);
  return 1;
}

int launch_preprocess_bwd(int app, const PreprocessBwdArgs &a, const CamDev &cam, cudaStream_t st, bool flags_ready) {
  if (app == GS_APP_SH) {
    if (a.n == 0) return 0;
    opt_in_smem(k_preprocess_bwd<GS_APP_SH>, kBwdSmemSH);
    launch_chained(k_preprocess_bwd<GS_APP_SH>, grid_for(a.n), kBlock, kBwdSmemSH, st, a, cam);
    return 1;
  } else if (app == GS_APP_SV) {
    if (a.n == 0) return 0;
    opt_in_smem(k_preprocess_bwd<GS_APP_SV>, kBwdSmemSV);
    launch_chained(k_preprocess_bwd<GS_APP_SV>, grid_for(a.n), kBlock, kBwdSmemSV, st, a, cam);
    return 1;
  } else if (app == kAppExternal) {
    if (a.n == 0) return 0;
    if (!flags_ready) launch_bwd_flags(a, false, st);
    const int wave = resident_blocks<k_preprocess_bwd_sparse<kAppExternal>>(sizeof(mlp::Weights), 1 << 20), chunks = grid_for(a.n);
    launch_chained(k_preprocess_bwd_sparse<kAppExternal>, chunks < wave ? chunks : wave, kBlock, sizeof(mlp::Weights), st, a, cam);
    return flags_ready ? 1 : 2;
  } else {
    if (app == kAppNeuralHalf) {
      opt_in_smem(k_preprocess_bwd_sparse<kAppNeuralHalf>, kBwdSmemNN);
      const int blocks = resident_blocks<k_preprocess_bwd_sparse<kAppNeuralHalf>>(kBwdSmemNN);
      if (a.n > 0) launch_chained(k_bwd_flags<true, true>, (int)((a.n + kFlagThreads - 1) / kFlagThreads), kFlagThreads, 0, st, a);
      launch_chained(k_preprocess_bwd_sparse<kAppNeuralHalf>, blocks, kBlock, kBwdSmemNN, st, a, cam);
      launch_wgrad_reduce(a.w_partials, blocks, a.g_weights, st);
      return 3;
    }
    opt_in_smem(k_preprocess_bwd_sparse<GS_APP_NEURAL>, kBwdSmemNN);
    const int blocks = resident_blocks<k_preprocess_bwd_sparse<GS_APP_NEURAL>>(kBwdSmemNN);
    if (a.n > 0) launch_chained(k_bwd_flags<true, true>, (int)((a.n + kFlagThreads - 1) / kFlagThreads), kFlagThreads, 0, st, a);
    launch_chained(k_preprocess_bwd_sparse<GS_APP_NEURAL>, blocks, kBlock, kBwdSmemNN, st, a, cam);
    launch_wgrad_reduce(a.w_partials, blocks, a.g_weights, st);
    return 3;
  }
}

template <int APP, bool BWD>
int launch_bulk(const AppearanceArgs &a, cudaStream_t st) {
  constexpr size_t smem = bulk_smem_bytes<APP>();
  opt_in_smem(k_appearance_bulk<APP, BWD>, smem);
  const int wave = resident_blocks<k_appearance_bulk<APP, BWD>>(smem), chunks = grid_for(a.n);
  k_appearance_bulk<APP, BWD><<<chunks < wave ? chunks : wave, kBlock, smem, st>>>(a);
  return 1;
}

// Grid of the tcgen05 kernel: tc::kCtasPerSm CTAs per SM.  The occupancy query answers 1 for this kernel, so the
// count is set here.
static int tc_wave() {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  return tc::kCtasPerSm * sms;
}

int launch_appearance_fwd(int app, const AppearanceArgs &a, cudaStream_t st) {
  if (a.n == 0) return 0;
  if (app == GS_APP_SH) return launch_bulk<GS_APP_SH, false>(a, st);
  if (app == GS_APP_SV) return launch_bulk<GS_APP_SV, false>(a, st);
  const int chunks = grid_for(a.n);
  // the tensor-memory path (tiles of 128 Gaussians = kBlock): on request, and by default from 2M Gaussians on, where it
  // measured 4-8 % faster than the warp-level kernel (at 1M it is 6-14 % slower: seven tiles per CTA do not pay for
  // staging the weights and allocating tensor memory)
  if (a.deg > 0 && (a.engine == GS_ENGINE_TCGEN05 || (a.engine == GS_ENGINE_AUTO && a.n >= 2000000))) {
    constexpr size_t smem = sizeof(tc::Smem);
    if (app == kAppNeuralHalf) {
      const int wave = tc_wave();
      tc::k_appearance_fwd_tc<false><<<chunks < wave ? chunks : wave, kBlock, smem, st>>>(a);
    } else {
      const int wave = tc_wave();
      tc::k_appearance_fwd_tc<true><<<chunks < wave ? chunks : wave, kBlock, smem, st>>>(a);
    }
    return 1;
  }
  if (app == kAppNeuralHalf) {
    const int wave = resident_blocks<k_appearance_fwd<kAppNeuralHalf>>(0, 1 << 20);
    k_appearance_fwd<kAppNeuralHalf><<<chunks < wave ? chunks : wave, kBlock, 0, st>>>(a);
  } else {
    const int wave = resident_blocks<k_appearance_fwd<GS_APP_NEURAL>>(0, 1 << 20);
    k_appearance_fwd<GS_APP_NEURAL><<<chunks < wave ? chunks : wave, kBlock, 0, st>>>(a);
  }
  return 1;
}

int launch_appearance_bwd(int app, const AppearanceArgs &a, cudaStream_t st) {
  if (app == GS_APP_SH) {
    if (a.n == 0) return 0;
    return launch_bulk<GS_APP_SH, true>(a, st);
  } else if (app == GS_APP_SV) {
    if (a.n == 0) return 0;
    return launch_bulk<GS_APP_SV, true>(a, st);
  } else {
    // the tensor-memory path: on request, and by default for split operands (measured 16-21 % faster than the
    // warp-level kernel from 1M to 10M Gaussians; with plain fp16 operands it is 6-9 % slower)
    if ((a.engine == GS_ENGINE_TCGEN05 || (a.engine == GS_ENGINE_AUTO && app != kAppNeuralHalf)) && a.deg > 0 && a.n > 0) {
      constexpr size_t smem = sizeof(tc::SmemBwd);
      int dev = 0, sms = 0;
      cudaGetDevice(&dev);
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
      int blocks = tc::kCtasPerSmBwd * sms;
      if (blocks > kWgradBlocks) blocks = kWgradBlocks;
      if (blocks > grid_for(a.n)) blocks = grid_for(a.n);
      if (app == kAppNeuralHalf) {
        opt_in_smem(tc::k_appearance_bwd_tc<false>, smem);
        tc::k_appearance_bwd_tc<false><<<blocks, kBlock, smem, st>>>(a);
      } else {
        opt_in_smem(tc::k_appearance_bwd_tc<true>, smem);
        tc::k_appearance_bwd_tc<true><<<blocks, kBlock, smem, st>>>(a);
      }
      launch_wgrad_reduce(a.w_partials, blocks, a.g_weights, st);
      return 2;
    }
    if (app == kAppNeuralHalf) {
      opt_in_smem(k_appearance_bwd<kAppNeuralHalf>, kBwdSmemNN);
      const int blocks = resident_blocks<k_appearance_bwd<kAppNeuralHalf>>(kBwdSmemNN);
      k_appearance_bwd<kAppNeuralHalf><<<blocks, kBlock, kBwdSmemNN, st>>>(a);
      launch_wgrad_reduce(a.w_partials, blocks, a.g_weights, st);
      return 2;
    }
    opt_in_smem(k_appearance_bwd<GS_APP_NEURAL>, kBwdSmemNN);
    const int blocks = resident_blocks<k_appearance_bwd<GS_APP_NEURAL>>(kBwdSmemNN);
    k_appearance_bwd<GS_APP_NEURAL><<<blocks, kBlock, kBwdSmemNN, st>>>(a);
    launch_wgrad_reduce(a.w_partials, blocks, a.g_weights, st);
    return 2;
  }
}

}  // namespace gs

// ---------------------------------------------------------------------------------------------
// gs_appearance_backward_noalloc: the neural appearance backward for callers that must not
// allocate.  Its only scratch, the per-block partial sums of the decoder-weight gradient, lives in
// the file-scope device array below instead of memory obtained from cudaMalloc.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kNoAllocChunksPerBlock = 32;                       // chunks of 128 Gaussians per CTA
constexpr int kNoAllocMaxBlocks = 1024;                          // rows of the static scratch
constexpr int64_t kNoAllocMaxN = (int64_t)kNoAllocMaxBlocks * kNoAllocChunksPerBlock * 128;   // 4,194,304
constexpr int kNoAllocMaxDevices = 64;
}  // namespace

// 1024 rows x 816 floats = 3,342,336 bytes, resident on every GPU that loads the library until the
// process exits.  Row b is written in full by CTA b of every launch before anything reads it, so no
// part of it has to start at zero; it keeps the previous call's values in between.
static __device__ __align__(256) float gs_noalloc_partials[kNoAllocMaxBlocks * GS_MLP_WEIGHTS];

extern "C" GsStatus gs_appearance_backward_noalloc(const GsScene *scene, const float *dirs, const float *dL_dcolor,
                                                   GsGrads *grads, float *dL_ddirs, void *stream, char *error_text,
                                                   size_t error_text_bytes) {
  using namespace gs;
  auto fail = [&](GsStatus code, const char *msg) {
    if (error_text && error_text_bytes) snprintf(error_text, error_text_bytes, "%s", msg);
    return code;
  };
  auto misaligned = [](const void *p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (!scene || !grads) return fail(GS_ERR_INVALID_ARG, "scene / grads is NULL");
  if (scene->app != GS_APP_NEURAL)
    return fail(GS_ERR_UNSUPPORTED, "only the neural appearance backward uses scratch memory; call gs_appearance_backward for SH");
  if (scene->active_degree < 0 || scene->active_degree > 3) return fail(GS_ERR_INVALID_ARG, "active_degree must be 0..3");
  if (scene->color_activation < GS_ACT_RELU || scene->color_activation > GS_ACT_HARD_SIGMOID)
    return fail(GS_ERR_INVALID_ARG, "unknown colour activation");
  if (scene->decoder_precision != GS_DECODER_SPLIT && scene->decoder_precision != GS_DECODER_HALF)
    return fail(GS_ERR_INVALID_ARG, "unknown decoder precision");
  if ((scene->mlp_hidden != 0 && scene->mlp_hidden != 16) || (scene->mlp_layers != 0 && scene->mlp_layers != 2) ||
      (scene->num_features != 0 && scene->num_features != 8))
    return fail(GS_ERR_UNSUPPORTED, "this entry point serves the 16 / 2 / 8 decoder only");
  if (scene->n < 0) return fail(GS_ERR_INVALID_ARG, "n < 0");
  if (scene->n > kNoAllocMaxN)
    return fail(GS_ERR_CAPACITY, "n exceeds 4194304 Gaussians, the most the static scratch of this entry point covers; "
                                 "split the call or use gs_appearance_backward");
  if (misaligned(grads->mlp_weights)) return fail(GS_ERR_INVALID_ARG, "grads->mlp_weights is NULL or misaligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (scene->n == 0) {
    if (cudaMemsetAsync(grads->mlp_weights, 0, sizeof(float) * GS_MLP_WEIGHTS, st) != cudaSuccess)
      return fail(GS_ERR_CUDA, "cudaMemsetAsync failed");
    return GS_OK;
  }
  if (misaligned(scene->base_color) || misaligned(scene->features) || misaligned(scene->mlp_weights) ||
      misaligned(dirs) || misaligned(dL_dcolor) || misaligned(dL_ddirs) || misaligned(grads->base_color) ||
      misaligned(grads->features))
    return fail(GS_ERR_INVALID_ARG, "an input or output pointer is NULL or not 16-byte aligned");

  // Set-up, once per device, with that device current: in host code the array's name is only a
  // stand-in for the symbol, so the kernel must be given the address the runtime reports for it.
  static float *scratch_of_device[kNoAllocMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices)
    return fail(GS_ERR_CUDA, "cudaGetDevice failed or device index >= 64");
  float *scratch = scratch_of_device[dev];
  if (!scratch) {
    void *p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, gs_noalloc_partials);
    if (e != cudaSuccess || !p) return fail(GS_ERR_CUDA, cudaGetErrorString(e));
    scratch = static_cast<float *>(p);
    scratch_of_device[dev] = scratch;      // same value from every thread, so a racing store is benign
  }

  AppearanceArgs a;
  memset(&a, 0, sizeof(a));
  a.n = scene->n; a.deg = scene->active_degree; a.act = scene->color_activation;
  a.base_color = scene->base_color; a.dirs = dirs;
  a.features = reinterpret_cast<const __half *>(scene->features);
  a.weights = reinterpret_cast<const __half *>(scene->mlp_weights);
  a.g_color = dL_dcolor;
  a.g_base = grads->base_color; a.g_features = grads->features; a.g_dirs = dL_ddirs;
  a.w_partials = scratch; a.g_weights = grads->mlp_weights;
  // one CTA per chunk of 128 Gaussians until the scratch's rows run out; from there on the CTAs walk the chunks with
  // the grid as their stride (at the largest n each covers 32 of them)
  const int64_t chunks = (a.n + kBlock - 1) / kBlock;
  const int blocks = (int)(chunks < kNoAllocMaxBlocks ? chunks : kNoAllocMaxBlocks);
  if (scene->decoder_precision == GS_DECODER_HALF) {   // same dispatch as gs_appearance_backward
    opt_in_smem(k_appearance_bwd<kAppNeuralHalf>, kBwdSmemNN);
    k_appearance_bwd<kAppNeuralHalf><<<blocks, kBlock, kBwdSmemNN, st>>>(a);
  } else {
    opt_in_smem(k_appearance_bwd<GS_APP_NEURAL>, kBwdSmemNN);
    k_appearance_bwd<GS_APP_NEURAL><<<blocks, kBlock, kBwdSmemNN, st>>>(a);
  }
  launch_wgrad_reduce(scratch, blocks, a.g_weights, st);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(GS_ERR_CUDA, cudaGetErrorString(e));
  return GS_OK;
}
