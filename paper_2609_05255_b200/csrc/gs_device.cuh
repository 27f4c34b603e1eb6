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
// Cells: 4 x 4 tiles.  The binning sorts one record per (Gaussian, cell) instead of one per (Gaussian, tile).
constexpr int kCellSlots = 9;                 // records kept per Gaussian by the preprocess (3 x 3 cells)
constexpr uint32_t kCellBig = 0x80000000u;    // flag in cell_count: records not stored, derive them again
constexpr int kCellChunk = 2048;              // records of one cell that one CTA expands

struct CamDev {
  int W, H, gx, gy;
  int cgx, cgy;         // cells per row / column: ceil(gx / 4), ceil(gy / 4)
  float fx, fy, cx, cy;
  float R[9], t[3];
  float oc[3];          // camera centre in world space
  float near_plane, far_plane;
  float limx, limy;     // 1.3 x half field of view, as tan
  float bg[3];
};

// ---- launches (all enqueue on `st`; none synchronises; each returns the number of kernels it
// launched) ---------------------------------------------------------------------------------
// Appearance "model" of the preprocess kernels in the separate-pass (unfused) step: no colour is decoded; the
// forward leaves the view directions of the visible Gaussians where the colours go, the backward takes dL/dd
// from a buffer.  The appearance kernels run as launches of their own around them.
constexpr int kAppExternal = 3;
// The neural model with the decoder's products taken on plain fp16 operands (the paper's precision) instead of
// split ones: GsScene.decoder_precision = GS_DECODER_HALF.  Same kernels, same weights, same layout.
constexpr int kAppNeuralHalf = 4;

struct PreprocessArgs {
  int64_t n;
  const float *means, *log_scales, *quats, *logits, *base_color, *sh_rest;
  const __half *features, *weights;
  int deg, act;
  float *mean2d, *conic_opacity, *color, *extent;
  uint32_t *depth_key, *tiles_touched, *cell_count, *cell_records;
  uint16_t *rect;
  unsigned long long *pair_counter;
};
int launch_preprocess_fwd(int app, const PreprocessArgs &a, const CamDev &cam, cudaStream_t st);

struct PreprocessBwdArgs {
  int64_t n;
  const float *means, *log_scales, *quats, *logits, *base_color, *sh_rest;
  const __half *features, *weights;
  int deg, act;
  const uint16_t *rect;
  const float *g2d;            // [n,12]: dL/dcolor(3), dL/dopacity, dL/dconic(3), dL/dmean2d(2), pad
  unsigned long long *timeout; // set to 1 if a bounded wait on a bulk copy ran out (never expected)
  const float *gd_in;          // kAppExternal only: [n,3] dL/dd from the separate appearance backward
  uint32_t *flags;             // scratch, one bit per Gaussian: it received a gradient in this view
  int nfeat;                   // features per Gaussian of g_features (8, or 16 for the raw-feature decoder variants)
  float *g_means, *g_log_scales, *g_quats, *g_logits, *g_base, *g_sh_rest, *g_features;
  float *w_partials;           // [kWgradBlocks, 816]
  float *g_weights;            // [816]
};
// flags_ready (kAppExternal): launch_bwd_flags has run on these arguments already.
int launch_preprocess_bwd(int app, const PreprocessBwdArgs &a, const CamDev &cam, cudaStream_t st, bool flags_ready = false);
// The flag bits (who received a gradient) and the zero rows of everyone else: projection gradients, and with
// appearance_rows also base colour and features.
int launch_bwd_flags(const PreprocessBwdArgs &a, bool appearance_rows, cudaStream_t st);

struct AppearanceArgs {
  int64_t n;
  int deg, act;
  const float *base_color, *sh_rest, *dirs;
  const __half *features, *weights;
  float *color;                // forward
  const float *g_color;        // backward
  float *g_base, *g_sh_rest, *g_features, *g_dirs;
  float *w_partials, *g_weights;
  unsigned long long *timeout; // optional: set to 1 if a bounded wait on a bulk copy ran out (never expected)
  int engine;                  // GsDecoderEngine for the default neural decoder: warp-level MMA, tcgen05, or per kernel the faster
  const uint32_t *mask;        // optional [n]: Gaussians with a zero here are skipped (no colour written; zero
                               // gradient rows written); the tiles-touched array in the unfused step
  const uint32_t *flags;       // optional, backward of the decoder variants on tcgen05: one bit per Gaussian; only the
                               // flagged ones are worked on (gathered into full tiles) and written
  const float *means, *g2d;    // optional, with flags (the unfused step): view directions from the means and the camera
  float oc[3];                 // centre oc, dL/dcolor from columns 0..2 of the [n,12] rows g2d, instead of dirs / g_color
};
int launch_appearance_fwd(int app, const AppearanceArgs &a, cudaStream_t st);
int launch_appearance_bwd(int app, const AppearanceArgs &a, cudaStream_t st);

// Decoder variants (1-3 hidden layers of 16 or 32 neurons, 8 encoded or 16 raw features): tcgen05 kernels unless
// a.engine is GS_ENGINE_WARP_MMA or the active degree is 0, fp32 FMA kernels then.
int variant_num_weights(int hidden, int layers);
size_t variant_partials_floats();   // floats of per-block weight-gradient partials the backward needs
int launch_variant_fwd(int hidden, int layers, int nfeat, const AppearanceArgs &a, cudaStream_t st);
int launch_variant_bwd(int hidden, int layers, int nfeat, const AppearanceArgs &a, cudaStream_t st);

// Unfused step, backward: view directions of the masked-in Gaussians and their dL/dcolor (columns 0..2 of the
// [n,12] rows) as dense [n,3] arrays for the separate appearance backward.
int launch_unfused_prepare(int64_t n, const float *means, const CamDev &cam, const float *g2d, const uint32_t *mask,
                           float *dirs, float *g_color, cudaStream_t st);

constexpr int kWgradBlocks = 592;   // persistent blocks of the decoder-gradient kernels (4 x 148)

// Sorting / binning.
// What the scatter of the last pass of a sort adds on its way out (nothing where the pointers are null).
struct SortEpilogue {
  // depth sort: sums of a per-Gaussian count (counts[id] & count_mask) per 256 consecutive Gaussians of the sorted
  // order, from which the record emission takes its offsets; cleared by the same pass
  const uint32_t *counts;
  uint32_t count_mask;
  uint32_t *block_sums;
  int num_block_sums;
  // record sort: [start, end) of every id = key >> key_shift in the sorted list (an id that does not occur is left at
  // (0xffffffff, 0)), and the flag raised when the device-side count exceeded the capacity
  uint32_t *ranges;
  int num_ranges;
  int key_shift;
  uint32_t *overflow;
};
size_t sort_scratch_bytes(int64_t count);
// LSD radix sort of (key, val) pairs on bits [first_bit, first_bit + num_bits), in digits of at most max_digit_bits
// (4 .. 11; wide digits save passes but take registers and shared memory: they pay for short keys only).  If vals_in == nullptr the values are
// the element indices.  Result lands in keys_out / vals_out; tmp_* are same-sized alternates.  `count` bounds the
// number of elements (and sizes the grid); with count_dev the true number is read on the device.
int launch_radix_sort(const uint32_t *keys_in, const uint32_t *vals_in, uint32_t *keys_out,
                       uint32_t *vals_out, uint32_t *tmp_keys, uint32_t *tmp_vals, int64_t count,
                       const unsigned long long *count_dev, int first_bit, int num_bits, int max_digit_bits, void *scratch,
                       const SortEpilogue *epilogue, cudaStream_t st);
int radix_passes(int num_bits, int max_digit_bits);   // passes launch_radix_sort makes over num_bits key bits
size_t scan_scratch_bytes(int64_t n);
int num_scan_blocks(int64_t n);   // entries of the block sums that launch_emit_records reads
int launch_emit_records(const uint32_t *depth_order, const uint32_t *cell_count, const uint32_t *cell_records,
                        const uint16_t *rect, const float *mean2d, const float *conic_opacity, const uint32_t *block_sums,
                        uint32_t *rec_keys, uint32_t *rec_vals, unsigned long long *rec_total, uint32_t *overflow, int64_t n,
                        int cgx, int W, int H, int64_t capacity, cudaStream_t st);
// Scratch of the expansion: chunk_first [cells + 1], chunk_counts and chunk_bases [max_chunks, 16], tile_counts and
// tile_starts [tiles].
struct CellScratch { uint32_t *chunk_first, *chunk_counts, *chunk_bases, *tile_counts, *tile_starts; };
int max_chunks(int64_t record_capacity, int num_cells);
int launch_expand(const uint32_t *rec_keys, const uint32_t *rec_vals, const uint32_t *cell_ranges, const CellScratch &cs,
                  int64_t record_capacity, int64_t pair_capacity, int gx, int gy, int cgx, int cgy,
                  uint32_t *sorted_vals, uint32_t *tile_ranges, uint32_t *tile_order, cudaStream_t st);
int launch_empty_binning(uint32_t *tile_ranges, uint32_t *tile_order, int num_tiles, cudaStream_t st);
void launch_flag_if_greater(const unsigned long long *value, unsigned long long bound, uint32_t *flag, cudaStream_t st);

// Blend.
// (sorted_tiles: the tile id of every instance of the sorted list, written by the tile's CTA on its way in)
int launch_blend_fwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                      const float *mean2d, const float *conic_opacity, const float *color, uint32_t *sorted_tiles,
                      float *image, float *final_T, uint32_t *n_contrib, cudaStream_t st);
int launch_blend_bwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                      const float *mean2d, const float *conic_opacity, const float *color,
                      const float *final_T, const uint32_t *n_contrib, const float *dL_dimage,
                      float *g2d, cudaStream_t st);

int launch_neural_fold(int64_t n, const __half *features, const __half *weights, __half *preact, cudaStream_t st);
int launch_neural_prepass(int64_t n, int deg, int act, const float *means, const float *logits, const float *base_color,
                          const __half *preact, const __half *weights, const float eye[3], uint8_t *rgba, float *color,
                          cudaStream_t st);
int launch_adam(const GsAdamTensor *tensors, int num_tensors, int64_t step, int num_sms, cudaStream_t st);
int launch_blend_count(const CamDev &cam, const uint32_t *ranges, const uint32_t *vals, const float *mean2d,
                       const float *conic_opacity, const float *color, unsigned long long *counts, cudaStream_t st);

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

// tau = 2 ln(255 o): the alpha >= 1/255 ellipse is conic-form <= tau.  One function, so that the
// preprocess and the instance emission get identical bits.
__device__ __forceinline__ float footprint_tau(float o) { return 2.f * logf(255.f * o); }

// Exact tile overlap of the alpha >= 1/255 ellipse, row of tiles by row of tiles.  The ellipse is
// (la dx + lb dy)^2 + (lc dy)^2 <= tau with (la, lb, lc) the Cholesky factor of the conic.  Over a
// band of pixel-centre rows dy in [da, db] the set is convex, so the tiles it meets in that row are
// exactly those between its leftmost and rightmost point; the rightmost point over the band is at
// the band end nearest to dy_r = -lb sqrt(tau / C) / lc (C = lb^2 + lc^2), the leftmost at the one
// nearest to -dy_r.  Every operation is rounded once, in a fixed order (no contraction), so the
// same integers come out of any IEEE fp32 evaluation; tau and the band are padded by 2e-5 / 1e-5
// so that rounding can only add a tile, never drop a pixel the blend would accept.
struct TileSpans {
  float u, v, ila, lb, lc, taup, dys, eyp;
  int W, H;
  __device__ __forceinline__ void setup(float u_, float v_, float la, float lb_, float lc_, float tau, int W_, int H_) {
    u = u_; v = v_; lb = lb_; lc = lc_; W = W_; H = H_;
    taup = __fmul_rn(tau, 1.00002f);
    const float rl = __frcp_rn(lc);
    ila = __frcp_rn(la);
    const float C = __fadd_rn(__fmul_rn(lb, lb), __fmul_rn(lc, lc));
    dys = __fmul_rn(__fmul_rn(lb, rl), __fsqrt_rn(__fdiv_rn(taup, C)));
    eyp = __fmul_rn(__fmul_rn(__fsqrt_rn(taup), rl), 1.00001f);
  }
  // Tiles [xa, xb) of tile row ty, clipped to the bounding rectangle's columns [tx0, tx1).
  __device__ __forceinline__ bool row(int ty, int tx0, int tx1, int &xa, int &xb) const {
    const float ylo = (float)(16 * ty) + 0.5f, yhi = fminf((float)(16 * ty) + 15.5f, (float)H - 0.5f);
    const float da = fmaxf(__fsub_rn(ylo, v), -eyp), db = fminf(__fsub_rn(yhi, v), eyp);
    if (!(da <= db)) return false;
    const float dyR = fminf(fmaxf(-dys, da), db), dyL = fminf(fmaxf(dys, da), db);
    const float tR = __fmul_rn(lc, dyR), tL = __fmul_rn(lc, dyL);
    const float sR = __fsqrt_rn(fmaxf(__fsub_rn(taup, __fmul_rn(tR, tR)), 0.f));
    const float sL = __fsqrt_rn(fmaxf(__fsub_rn(taup, __fmul_rn(tL, tL)), 0.f));
    const float xr = __fmul_rn(__fsub_rn(sR, __fmul_rn(lb, dyR)), ila);
    const float xl = __fmul_rn(__fsub_rn(-sL, __fmul_rn(lb, dyL)), ila);
    const float ihi = floorf(__fsub_rn(__fadd_rn(u, xr), 0.5f)), ilo = ceilf(__fsub_rn(__fadd_rn(u, xl), 0.5f));
    if (!(ilo <= ihi) || ihi < 0.f || ilo > (float)(W - 1)) return false;
    const int pa = (int)fmaxf(ilo, 0.f), pb = (int)fminf(ihi, (float)(W - 1));
    xa = max(pa >> 4, tx0);
    xb = min((pb >> 4) + 1, tx1);
    return xa < xb;
  }
  __device__ __forceinline__ unsigned count(int tx0, int ty0, int tx1, int ty1) const {
    unsigned c = 0;
    for (int ty = ty0; ty < ty1; ++ty) {
      int xa, xb;
      if (row(ty, tx0, tx1, xa, xb)) c += (unsigned)(xb - xa);
    }
    return c;
  }
};

// Colour activations (Sec. 3.1) of z = c0 + 0.5 + A(d) and their derivatives: 0 ReLU(z), 1 softplus(z) with
// beta = 10, 2 sigmoid(4 (z - 0.5)), 3 clamp(z, 0, 1).  The derivative at a kink is 0.
__device__ __forceinline__ float color_act_z(int act, float z) {
  if (act == GS_ACT_SOFTPLUS) { const float t = 10.f * z; return t > 15.f ? z : 0.1f * log1pf(expf(t)); }
  if (act == GS_ACT_SIGMOID) return 1.f / (1.f + expf(fmaf(-4.f, z, 2.f)));
  if (act == GS_ACT_HARD_SIGMOID) return fminf(fmaxf(z, 0.f), 1.f);
  return fmaxf(z, 0.f);
}
__device__ __forceinline__ float color_act_grad_z(int act, float z) {
  if (act == GS_ACT_SOFTPLUS) return 1.f / (1.f + expf(-10.f * z));
  if (act == GS_ACT_SIGMOID) { const float y = 1.f / (1.f + expf(fmaf(-4.f, z, 2.f))); return 4.f * y * (1.f - y); }
  if (act == GS_ACT_HARD_SIGMOID) return (z > 0.f && z < 1.f) ? 1.f : 0.f;
  return z > 0.f ? 1.f : 0.f;
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- the neural decoder's inputs and residual squashing, shared by every kernel that evaluates it
__device__ __forceinline__ void unpack_features(const uint4 &raw, float f[8]) {
  const __half2 *h = reinterpret_cast<const __half2 *>(&raw);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 v = __half22float2(h[j]);
    f[2 * j] = v.x; f[2 * j + 1] = v.y;
  }
}
__device__ __forceinline__ void load_features(const __half *features, int64_t i, float f[8]) {
  unpack_features(__ldg(reinterpret_cast<const uint4 *>(features) + i), f);
}

// Decoder inputs of one Gaussian (Eq. 5, Eq. 6 with k = 1): SH basis of the direction masked by the
// active degree, then (sin f_j, cos f_j).  The fast sincos is used inside [-pi, pi] (absolute error
// below 4e-7 there), the accurate one outside.
__device__ __forceinline__ void decoder_inputs(float dx, float dy, float dz, const float f[8], int deg, float x[32]) {
  sh_basis(dx, dy, dz, x);
  const int na = (deg + 1) * (deg + 1);
  if (na < 16) {
#pragma unroll
    for (int k = 0; k < 16; ++k) x[k] = k < na ? x[k] : 0.f;
  }
  float big = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) big = fmaxf(big, fabsf(f[j]));
  if (big <= 3.14159265f) {   // one decision for the eight of them: features are O(0.1 .. 1)
#pragma unroll
    for (int j = 0; j < 8; ++j) __sincosf(f[j], &x[16 + 2 * j], &x[17 + 2 * j]);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) sincosf(f[j], &x[16 + 2 * j], &x[17 + 2 * j]);
  }
}

// tanh(y) = 1 - 2 / (e^{2y} + 1) on the exponential and reciprocal units: absolute error of a few 1e-7 over the
// whole range (the residual is an absolute colour offset, so that is the error that counts), saturating to +-1.
__device__ __forceinline__ float tanh_fast(float y) {
  const float e = ex2_approx(y * 2.885390081777927f);    // 2 log2(e)
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.f));
  return fmaf(-2.f, r, 1.f);
}

// Programmatic dependent launch.  The kernels of the binning (gs_sort.cu) form chains of short, dependent launches (27 per view).
// Launched with the attribute below, a kernel may be placed on the SMs as soon as the CTAs of its predecessor in the
// stream have exited, without waiting for the predecessor's completion to be processed; dependency_wait() returns once
// the predecessor has completed and its writes are visible, and every kernel here calls it before its first access to
// global memory, so the order of all reads and writes is the stream's.  Launched without the attribute it is a no-op.
// Measured on one stream: 214 instead of 248 us of binning per view.  Letting the successor in earlier
// (griddepcontrol.launch_dependents at the top of every kernel) gained no more on one stream and cost 4 % with
// several views in flight: the successor's CTAs then sit on the SMs for the whole run of the predecessor, in the
// places of the other streams' kernels.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <class... KArgs, class... Args>
void launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#endif  // __CUDACC__

}  // namespace gs
