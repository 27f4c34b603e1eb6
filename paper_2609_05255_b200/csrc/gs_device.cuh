// Internal declarations shared by the translation units of libgs_b200 (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "gs.h"

namespace gs {

constexpr float kAlphaMin = 1.0f / 255.0f;
constexpr float kAlphaMax = 0.99f;
constexpr float kTmin = 1e-4f;
constexpr float kDilation = 0.3f;
constexpr float kExtentPad = 1.00001f;  // keeps fp32 rounding from dropping an edge pixel
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMlpW1 = 0, kMlpW2 = 512, kMlpW3 = 768;

// Camera as the kernels see it (passed by value).
struct CamDev {
  int W, H, gx, gy;
  float fx, fy, cx, cy;
  float R[9], t[3];
  float oc[3];          // camera centre in world space
  float near_plane, far_plane;
  float limx, limy;     // 1.3 x half field of view, as tan
  float bg[3];
};

// ---- launches (all enqueue on `st`; none synchronises; each returns the number of kernels it
// launched) ---------------------------------------------------------------------------------
struct PreprocessArgs {
  int64_t n;
  const float *means, *log_scales, *quats, *logits, *base_color, *sh_rest;
  const __half *features, *weights;
  int deg;
  float *mean2d, *conic_opacity, *color, *extent;
  uint32_t *depth_key;
  uint16_t *rect;
  unsigned long long *pair_counter;
};
int launch_preprocess_fwd(int app, const PreprocessArgs &a, const CamDev &cam, cudaStream_t st);

struct PreprocessBwdArgs {
  int64_t n;
  const float *means, *log_scales, *quats, *logits, *base_color, *sh_rest;
  const __half *features, *weights;
  int deg;
  const uint16_t *rect;
  const float *g2d;            // [n,12]: dL/dcolor(3), dL/dopacity, dL/dconic(3), dL/dmean2d(2), pad
  float *g_means, *g_log_scales, *g_quats, *g_logits, *g_base, *g_sh_rest, *g_features;
  float *w_partials;           // [kWgradBlocks, 816]
  float *g_weights;            // [816]
};
int launch_preprocess_bwd(int app, const PreprocessBwdArgs &a, const CamDev &cam, cudaStream_t st);

struct AppearanceArgs {
  int64_t n;
  int deg;
  const float *base_color, *sh_rest, *dirs;
  const __half *features, *weights;
  float *color;                // forward
  const float *g_color;        // backward
  float *g_base, *g_sh_rest, *g_features, *g_dirs;
  float *w_partials, *g_weights;
};
int launch_appearance_fwd(int app, const AppearanceArgs &a, cudaStream_t st);
int launch_appearance_bwd(int app, const AppearanceArgs &a, cudaStream_t st);

constexpr int kWgradBlocks = 592;   // persistent blocks of the decoder-gradient kernels (4 x 148)

// Sorting / binning.
size_t sort_scratch_bytes(int64_t count);
// LSD radix sort of (key, val) pairs on bits [0, num_bits).  If vals_in == nullptr the values are
// the element indices.  Result lands in keys_out / vals_out; tmp_* are same-sized alternates.
int launch_radix_sort(const uint32_t *keys_in, const uint32_t *vals_in, uint32_t *keys_out,
                       uint32_t *vals_out, uint32_t *tmp_keys, uint32_t *tmp_vals, int64_t count,
                       int num_bits, void *scratch, cudaStream_t st);
size_t scan_scratch_bytes(int64_t n);
int launch_tile_offsets(const uint32_t *depth_order, const uint16_t *rect, uint32_t *offsets,
                         int64_t n, void *scratch, cudaStream_t st);
int launch_keygen(const uint32_t *depth_order, const uint16_t *rect, const uint32_t *offsets,
                   uint32_t *inst_tiles, uint32_t *inst_vals, int64_t n, int gx, cudaStream_t st);
int launch_tile_ranges(const uint32_t *sorted_tiles, int64_t P, uint32_t *ranges, uint32_t *order,
                       int num_tiles, cudaStream_t st);

// Blend.
int launch_blend_fwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                      const float *mean2d, const float *conic_opacity, const float *color,
                      float *image, float *final_T, uint32_t *n_contrib, cudaStream_t st);
int launch_blend_bwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                      const float *mean2d, const float *conic_opacity, const float *color,
                      const float *final_T, const uint32_t *n_contrib, const float *dL_dimage,
                      float *g2d, cudaStream_t st);

// ---- device helpers -------------------------------------------------------------------------
#ifdef __CUDACC__

// Real orthonormal SH basis, degrees 0..3, order m = -l..l.
__device__ __forceinline__ void sh_basis(float x, float y, float z, float Y[16]) {
  const float xx = x * x, yy = y * y, zz = z * z;
  Y[0] = 0.28209479177387814f;
  Y[1] = -0.4886025119029199f * y;
  Y[2] = 0.4886025119029199f * z;
  Y[3] = -0.4886025119029199f * x;
  Y[4] = 1.0925484305920792f * x * y;
  Y[5] = -1.0925484305920792f * y * z;
  Y[6] = 0.31539156525252005f * (2.f * zz - xx - yy);
  Y[7] = -1.0925484305920792f * x * z;
  Y[8] = 0.5462742152960396f * (xx - yy);
  Y[9] = -0.5900435899266435f * y * (3.f * xx - yy);
  Y[10] = 2.890611442640554f * x * y * z;
  Y[11] = -0.4570457994644658f * y * (4.f * zz - xx - yy);
  Y[12] = 0.3731763325901154f * z * (2.f * zz - 3.f * xx - 3.f * yy);
  Y[13] = -0.4570457994644658f * x * (4.f * zz - xx - yy);
  Y[14] = 1.445305721320277f * z * (xx - yy);
  Y[15] = -0.5900435899266435f * x * (xx - 3.f * yy);
}

// Accumulate g_d += w * grad Y_k(d) for one basis function (k is a compile-time constant after
// unrolling).
__device__ __forceinline__ void sh_grad_acc(int k, float x, float y, float z, float w, float &gx,
                                            float &gy, float &gz) {
  const float c1 = 0.4886025119029199f, c2a = 1.0925484305920792f, c2b = 0.31539156525252005f,
              c2c = 0.5462742152960396f, c3a = 0.5900435899266435f, c3b = 2.890611442640554f,
              c3c = 0.4570457994644658f, c3d = 0.3731763325901154f, c3e = 1.445305721320277f;
  switch (k) {
    case 1: gy -= c1 * w; break;
    case 2: gz += c1 * w; break;
    case 3: gx -= c1 * w; break;
    case 4: gx += c2a * y * w; gy += c2a * x * w; break;
    case 5: gy -= c2a * z * w; gz -= c2a * y * w; break;
    case 6: gx -= 2.f * c2b * x * w; gy -= 2.f * c2b * y * w; gz += 4.f * c2b * z * w; break;
    case 7: gx -= c2a * z * w; gz -= c2a * x * w; break;
    case 8: gx += 2.f * c2c * x * w; gy -= 2.f * c2c * y * w; break;
    case 9: gx -= 6.f * c3a * x * y * w; gy -= 3.f * c3a * (x * x - y * y) * w; break;
    case 10: gx += c3b * y * z * w; gy += c3b * x * z * w; gz += c3b * x * y * w; break;
    case 11: gx += 2.f * c3c * x * y * w; gy -= c3c * (4.f * z * z - x * x - 3.f * y * y) * w;
             gz -= 8.f * c3c * y * z * w; break;
    case 12: gx -= 6.f * c3d * x * z * w; gy -= 6.f * c3d * y * z * w;
             gz += 3.f * c3d * (2.f * z * z - x * x - y * y) * w; break;
    case 13: gx -= c3c * (4.f * z * z - 3.f * x * x - y * y) * w; gy += 2.f * c3c * x * y * w;
             gz -= 8.f * c3c * x * z * w; break;
    case 14: gx += 2.f * c3e * x * z * w; gy -= 2.f * c3e * y * z * w; gz += c3e * (x * x - y * y) * w; break;
    case 15: gx -= 3.f * c3a * (x * x - y * y) * w; gy += 6.f * c3a * x * y * w; break;
    default: break;
  }
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One pixel-Gaussian evaluation, shared by the forward and the backward blend so that both
// take identical skip decisions.  q = (-0.5 A log2e, -B log2e, -0.5 C log2e).  Returns false if
// the pair is skipped; e2 = exp(power), alpha = min(0.99, o * e2).
__device__ __forceinline__ bool eval_alpha(float dx, float dy, float qa, float qb, float qc, float o,
                                           float &e2, float &alpha) {
  const float p = __fmaf_rn(__fmaf_rn(qa, dx, __fmul_rn(qb, dy)), dx, __fmul_rn(__fmul_rn(qc, dy), dy));
  if (p > 0.f) return false;
  e2 = ex2_approx(p);
  alpha = fminf(kAlphaMax, __fmul_rn(o, e2));
  return alpha >= kAlphaMin;
}

#endif  // __CUDACC__

}  // namespace gs
