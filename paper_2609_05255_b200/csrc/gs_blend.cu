// Per-tile alpha blending, forward and backward.  One CTA of 64 threads per 16x16 tile; every
// thread owns a 2x2 pixel quad (a warp covers 16x8 pixels), so one shared-memory read of a
// Gaussian serves four pixels and, in the backward, four pixels are summed in registers before
// anything crosses lanes.  The tile's depth-ordered instance list is staged through shared memory
// in batches of 128 Gaussians.
#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kThreads = 64;
constexpr int kBatch = 128;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kLn2 = 0.6931471805599453f;

// Top-left pixel of this thread's quad.
__device__ __forceinline__ void quad_of(int tile, int gx, int tid, int &px, int &py) {
  const int tx = tile % gx, ty = tile / gx;
  const int warp = tid >> 5, lane = tid & 31;
  px = tx * GS_TILE + 2 * (lane & 7);
  py = ty * GS_TILE + warp * 8 + 2 * (lane >> 3);
}

// Stage one batch entry: (x, y, la, lb) (lc, o) (r, g, b, -).  (la, lb, lc) is the Cholesky factor
// of the conic, scaled by sqrt(0.5 log2 e), so that exp(power) = 2^-((la dx + lb dy)^2 + (lc dy)^2):
// a sum of two squares has no cancellation, which keeps alpha accurate to a few ulp even for
// footprints hundreds of pixels wide (the expanded quadratic form loses 1e-4 there).
__device__ __forceinline__ void stage_entry(uint32_t g, const float *mean2d, const float *conic_opacity,
                                            const float *color, float4 &xyab, float2 &co, float4 &rgb) {
  const float2 m = __ldg(reinterpret_cast<const float2 *>(mean2d) + g);
  const float4 q = __ldg(reinterpret_cast<const float4 *>(conic_opacity) + g);
  const float kS = 0.8493218002880191f;   // sqrt(0.5 * log2(e))
  xyab = make_float4(m.x, m.y, kS * q.x, kS * q.y);   // q = (l11, l21, l22, opacity)
  co = make_float2(kS * q.z, q.w);
  rgb = make_float4(__ldg(color + 3 * (size_t)g), __ldg(color + 3 * (size_t)g + 1), __ldg(color + 3 * (size_t)g + 2), 0.f);
}

// log2 of the Gaussian falloff at the four pixels of a quad; dx0, dy0 are the offsets of the
// top-left pixel centre from the mean.  Index k = 2 * row + column.  One explicit operation order,
// shared by the forward and the backward so that both take identical skip decisions.
// t1[k] = la dx + lb dy is returned too: the backward needs it for the gradient of the mean.
__device__ __forceinline__ void quad_power(float dx0, float dy0, float la, float lb, float lc, float p[4],
                                           float t1[4], float t2[2]) {
  const float dx1 = __fadd_rn(dx0, 1.f), dy1 = __fadd_rn(dy0, 1.f);
  const float a0 = __fmul_rn(la, dx0), a1 = __fmul_rn(la, dx1);
  t2[0] = __fmul_rn(lc, dy0); t2[1] = __fmul_rn(lc, dy1);
  const float s0 = __fmul_rn(t2[0], t2[0]), s1 = __fmul_rn(t2[1], t2[1]);
  t1[0] = __fmaf_rn(lb, dy0, a0); t1[1] = __fmaf_rn(lb, dy0, a1);
  t1[2] = __fmaf_rn(lb, dy1, a0); t1[3] = __fmaf_rn(lb, dy1, a1);
  p[0] = -__fmaf_rn(t1[0], t1[0], s0); p[1] = -__fmaf_rn(t1[1], t1[1], s0);
  p[2] = -__fmaf_rn(t1[2], t1[2], s1); p[3] = -__fmaf_rn(t1[3], t1[3], s1);
}

// alpha of one pixel from its log2 falloff; false if the pair is skipped.
__device__ __forceinline__ bool alpha_of(float p, float o, float &e2, float &alpha) {
  e2 = ex2_approx(p);             // p <= 0 by construction
  alpha = fminf(kAlphaMax, __fmul_rn(o, e2));
  return alpha >= kAlphaMin;
}

__global__ void __launch_bounds__(kThreads) k_blend_fwd(CamDev cam, const uint32_t *__restrict__ ranges,
                                                        const uint32_t *__restrict__ order,
                                                        const uint32_t *__restrict__ vals,
                                                        const float *__restrict__ mean2d,
                                                        const float *__restrict__ conic_opacity,
                                                        const float *__restrict__ color, float *__restrict__ image,
                                                        float *__restrict__ final_T, uint32_t *__restrict__ n_contrib) {
  __shared__ float4 s_xyab[kBatch];
  __shared__ float2 s_co[kBatch];
  __shared__ float4 s_rgb[kBatch];
  const int tid = threadIdx.x, tile = (int)__ldg(order + blockIdx.x);
  int px, py;
  quad_of(tile, cam.gx, tid, px, py);
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  float T[4], Cr[4], Cg[4], Cb[4];
  uint32_t last[4];
  unsigned live = 0;   // bit k set while pixel k still composites
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    T[k] = 1.f; Cr[k] = Cg[k] = Cb[k] = 0.f; last[k] = 0;
    if (px + (k & 1) < cam.W && py + (k >> 1) < cam.H) live |= 1u << k;
  }
  for (uint32_t base = start; base < end; base += kBatch) {
    if (__syncthreads_and(live == 0)) break;
#pragma unroll
    for (int h = 0; h < kBatch / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      const uint32_t idx = base + slot;
      if (idx < end) stage_entry(__ldg(vals + idx), mean2d, conic_opacity, color, s_xyab[slot], s_co[slot], s_rgb[slot]);
    }
    __syncthreads();
    const int cnt = (int)min((uint32_t)kBatch, end - base);
    for (int j = 0; j < cnt && live; ++j) {
      const float4 a = s_xyab[j];
      const float2 c = s_co[j];
      float p[4], t1[4], t2[2];
      quad_power(fx - a.x, fy - a.y, a.z, a.w, c.x, p, t1, t2);
      const float4 col = s_rgb[j];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float e2, alpha;
        if (!((live >> k) & 1u) || !alpha_of(p[k], c.y, e2, alpha)) continue;
        const float Tn = __fmul_rn(T[k], 1.f - alpha);
        if (Tn < kTmin) { live &= ~(1u << k); continue; }
        const float w = __fmul_rn(alpha, T[k]);
        Cr[k] = fmaf(col.x, w, Cr[k]); Cg[k] = fmaf(col.y, w, Cg[k]); Cb[k] = fmaf(col.z, w, Cb[k]);
        T[k] = Tn;
        last[k] = base - start + (uint32_t)j + 1u;
      }
    }
  }
  const size_t plane = (size_t)cam.W * cam.H;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int x = px + (k & 1), y = py + (k >> 1);
    if (x < cam.W && y < cam.H) {
      const size_t pix = (size_t)y * cam.W + x;
      image[pix] = fmaf(T[k], cam.bg[0], Cr[k]);
      image[plane + pix] = fmaf(T[k], cam.bg[1], Cg[k]);
      image[2 * plane + pix] = fmaf(T[k], cam.bg[2], Cb[k]);
      final_T[pix] = T[k];
      n_contrib[pix] = last[k];
    }
  }
}

// Sum nine per-lane values over the warp with 14 shuffles instead of 45.  Values 0..7: at each of
// the first three butterfly levels a lane keeps only the half of the values it is "responsible"
// for and trades the other half with its partner, so the exchanged volume halves each level
// (4 + 2 + 1 shuffles); two plain levels finish the one value left per lane.  Afterwards the
// lanes 0, 4, .., 28 hold the totals: lane 16 * b4 + 8 * b3 + 4 * b2 owns value 4 * b4 + 2 * b3 + b2.
// Value 8 takes a plain five-level butterfly and ends in every lane.
__device__ __forceinline__ void warp_reduce9(const float v[9], int lane, float &mine, float &ninth) {
  float a[4], b[2], c;
  const bool hi16 = lane & 16, hi8 = lane & 8, hi4 = lane & 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float keep = hi16 ? v[4 + i] : v[i], give = hi16 ? v[i] : v[4 + i];
    a[i] = keep + __shfl_xor_sync(kFull, give, 16);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float keep = hi8 ? a[2 + i] : a[i], give = hi8 ? a[i] : a[2 + i];
    b[i] = keep + __shfl_xor_sync(kFull, give, 8);
  }
  {
    const float keep = hi4 ? b[1] : b[0], give = hi4 ? b[0] : b[1];
    c = keep + __shfl_xor_sync(kFull, give, 4);
  }
  c += __shfl_xor_sync(kFull, c, 2);
  c += __shfl_xor_sync(kFull, c, 1);
  mine = c;
  float n = v[8];
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(kFull, n, s);
  ninth = n;
}

// Backward: walk each pixel's composited entries back to front.  The transmittance in front of
// an entry is recovered by dividing out (1 - alpha); the light arriving from behind it is summed
// up on the way (both stay relatively accurate: a front-to-back replay that forms that light as
// "final pixel - prefix" cancels badly for deep entries).  The nine per-Gaussian partial
// derivatives are summed over the thread's four pixels in registers, over the warp with
// warp_reduce9, over the tile's two warps in shared memory, and leave with one global atomic per
// value.
// g2d row: (d colour r, g, b, d opacity) (d conic A, B, C, d mean u) (d mean v, -, -, -).  Inside
// the kernel the values travel as v[0..7] = (conic A, B, C, mean u, mean v, colour r, g, b) and
// v[8] = opacity.
__global__ void __launch_bounds__(kThreads) k_blend_bwd(CamDev cam, const uint32_t *__restrict__ ranges,
                                                        const uint32_t *__restrict__ order,
                                                        const uint32_t *__restrict__ vals,
                                                        const float *__restrict__ mean2d,
                                                        const float *__restrict__ conic_opacity,
                                                        const float *__restrict__ color,
                                                        const float *__restrict__ final_T,
                                                        const uint32_t *__restrict__ n_contrib,
                                                        const float *__restrict__ dL_dimage, float *__restrict__ g2d) {
  __shared__ float4 s_xyab[kBatch];
  __shared__ float2 s_co[kBatch];
  __shared__ float4 s_rgb[kBatch];
  __shared__ uint32_t s_gid[kBatch];
  __shared__ float s_acc[kBatch][9];
  __shared__ uint32_t s_max[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, tile = (int)__ldg(order + blockIdx.x);
  int px, py;
  quad_of(tile, cam.gx, tid, px, py);
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  const size_t plane = (size_t)cam.W * cam.H;
  uint32_t nc[4];
  float T[4], Gr[4], Gg[4], Gb[4], Sr[4], Sg[4], Sb[4];
  uint32_t wmax = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int x = px + (k & 1), y = py + (k >> 1);
    nc[k] = 0; T[k] = 1.f; Gr[k] = Gg[k] = Gb[k] = 0.f;
    if (x < cam.W && y < cam.H) {
      const size_t pix = (size_t)y * cam.W + x;
      nc[k] = __ldg(n_contrib + pix);
      T[k] = __ldg(final_T + pix);
      Gr[k] = __ldg(dL_dimage + pix); Gg[k] = __ldg(dL_dimage + plane + pix); Gb[k] = __ldg(dL_dimage + 2 * plane + pix);
    }
    Sr[k] = T[k] * cam.bg[0]; Sg[k] = T[k] * cam.bg[1]; Sb[k] = T[k] * cam.bg[2];
    wmax = max(wmax, nc[k]);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) wmax = max(wmax, __shfl_xor_sync(kFull, wmax, s));
  if (lane == 0) s_max[warp] = wmax;
  __syncthreads();
  const uint32_t maxc = max(s_max[0], s_max[1]);
  if (maxc == 0 || start + maxc > end) return;   // nothing composited in this tile
  // column of the g2d row that this lane's reduced value belongs to (lanes 0, 4, .., 28)
  const int my_value = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
  const int my_col = my_value < 5 ? my_value + 4 : my_value - 5;
  const int nbatches = (int)((maxc + kBatch - 1) / kBatch);
  for (int b = nbatches - 1; b >= 0; --b) {
    __syncthreads();
    const uint32_t first = (uint32_t)b * kBatch;
    const int cnt = (int)min((uint32_t)kBatch, maxc - first);
#pragma unroll
    for (int h = 0; h < kBatch / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      if (slot < cnt) {
        const uint32_t g = __ldg(vals + start + first + slot);
        s_gid[slot] = g;
        stage_entry(g, mean2d, conic_opacity, color, s_xyab[slot], s_co[slot], s_rgb[slot]);
      }
#pragma unroll
      for (int k = 0; k < 9; ++k) s_acc[slot][k] = 0.f;
    }
    __syncthreads();
    const int jtop = (int)min((uint32_t)cnt, wmax > first ? wmax - first : 0u);
    for (int j = jtop - 1; j >= 0; --j) {
      const uint32_t pos = first + (uint32_t)j;
      const float4 a = s_xyab[j];
      const float2 c = s_co[j];
      const float dx0 = fx - a.x, dy0 = fy - a.y;
      float p[4], t1[4], t2[2];
      quad_power(dx0, dy0, a.z, a.w, c.x, p, t1, t2);
      const float4 col = s_rgb[j];
      float v[9];
#pragma unroll
      for (int k = 0; k < 9; ++k) v[k] = 0.f;
      bool any = false;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float e2, alpha;
        if (pos >= nc[k] || !alpha_of(p[k], c.y, e2, alpha)) continue;
        any = true;
        const float dx = dx0 + (float)(k & 1), dy = dy0 + (float)(k >> 1);
        const float inv = __frcp_rn(1.f - alpha);
        const float Tb = T[k] * inv;              // transmittance in front of this entry
        const float w = alpha * Tb;
        v[5] = fmaf(w, Gr[k], v[5]); v[6] = fmaf(w, Gg[k], v[6]); v[7] = fmaf(w, Gb[k], v[7]);
        // d pixel / d alpha = T c - S / (1 - alpha), S = everything composited behind this entry
        const float dalpha = Gr[k] * (Tb * col.x - Sr[k] * inv) + Gg[k] * (Tb * col.y - Sg[k] * inv) +
                             Gb[k] * (Tb * col.z - Sb[k] * inv);
        if (c.y * e2 <= kAlphaMax) {              // not clamped: alpha depends on o and power
          v[8] = fmaf(e2, dalpha, v[8]);
          const float dp = alpha * dalpha;
          const float dp2 = dp * (2.f * kLn2);    // power = -ln2 (t1^2 + t2^2), d power / d mean = -d / d (dx, dy)
          v[0] = fmaf(-0.5f * dx * dx, dp, v[0]);
          v[1] = fmaf(-dx * dy, dp, v[1]);
          v[2] = fmaf(-0.5f * dy * dy, dp, v[2]);
          v[3] = fmaf(dp2, t1[k] * a.z, v[3]);
          v[4] = fmaf(dp2, fmaf(t1[k], a.w, t2[k >> 1] * c.x), v[4]);
        }
        Sr[k] = fmaf(col.x, w, Sr[k]); Sg[k] = fmaf(col.y, w, Sg[k]); Sb[k] = fmaf(col.z, w, Sb[k]);
        T[k] = Tb;
      }
      if (__any_sync(kFull, any)) {
        float mine, ninth;
        warp_reduce9(v, lane, mine, ninth);
        if ((lane & 3) == 0) atomicAdd(&s_acc[j][my_col], mine);
        if (lane == 1) atomicAdd(&s_acc[j][3], ninth);
      }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < kBatch / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      if (slot < cnt) {
        float *dst = g2d + (size_t)s_gid[slot] * 12;
        bool touched = false;
#pragma unroll
        for (int k = 0; k < 9; ++k) touched = touched || (s_acc[slot][k] != 0.f);
        if (touched) {
#pragma unroll
          for (int k = 0; k < 9; ++k) atomicAdd(dst + k, s_acc[slot][k]);
        }
      }
    }
  }
}

// Measurement only: replay the forward's decisions and count, over all pixels, the list entries
// evaluated (until each pixel stopped) and the pairs composited.  counts[0] += evaluated,
// counts[1] += composited.
__global__ void __launch_bounds__(kThreads) k_blend_count(CamDev cam, const uint32_t *__restrict__ ranges,
                                                          const uint32_t *__restrict__ vals,
                                                          const float *__restrict__ mean2d,
                                                          const float *__restrict__ conic_opacity,
                                                          const float *__restrict__ color,
                                                          unsigned long long *__restrict__ counts) {
  __shared__ float4 s_xyab[kBatch];
  __shared__ float2 s_co[kBatch];
  __shared__ float4 s_rgb[kBatch];
  const int tid = threadIdx.x, tile = blockIdx.x;
  int px, py;
  quad_of(tile, cam.gx, tid, px, py);
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  float T[4] = {1.f, 1.f, 1.f, 1.f};
  unsigned live = 0;
  unsigned long long evaluated = 0, composited = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k)
    if (px + (k & 1) < cam.W && py + (k >> 1) < cam.H) live |= 1u << k;
  for (uint32_t base = start; base < end; base += kBatch) {
    if (__syncthreads_and(live == 0)) break;
#pragma unroll
    for (int h = 0; h < kBatch / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      const uint32_t idx = base + slot;
      if (idx < end) stage_entry(__ldg(vals + idx), mean2d, conic_opacity, color, s_xyab[slot], s_co[slot], s_rgb[slot]);
    }
    __syncthreads();
    const int cnt = (int)min((uint32_t)kBatch, end - base);
    for (int j = 0; j < cnt && live; ++j) {
      const float4 a = s_xyab[j];
      const float2 c = s_co[j];
      float p[4], t1[4], t2[2];
      quad_power(fx - a.x, fy - a.y, a.z, a.w, c.x, p, t1, t2);
      evaluated += __popc(live);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float e2, alpha;
        if (!((live >> k) & 1u) || !alpha_of(p[k], c.y, e2, alpha)) continue;
        const float Tn = __fmul_rn(T[k], 1.f - alpha);
        if (Tn < kTmin) { live &= ~(1u << k); continue; }
        T[k] = Tn;
        ++composited;
      }
    }
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    evaluated += __shfl_xor_sync(kFull, evaluated, s);
    composited += __shfl_xor_sync(kFull, composited, s);
  }
  if ((tid & 31) == 0) { atomicAdd(counts, evaluated); atomicAdd(counts + 1, composited); }
}

}  // namespace

int launch_blend_count(const CamDev &cam, const uint32_t *ranges, const uint32_t *vals, const float *mean2d,
                       const float *conic_opacity, const float *color, unsigned long long *counts, cudaStream_t st) {
  k_blend_count<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, vals, mean2d, conic_opacity, color, counts);
  return 1;
}

int launch_blend_fwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                     const float *mean2d,
                     const float *conic_opacity, const float *color, float *image, float *final_T,
                     uint32_t *n_contrib, cudaStream_t st) {
  k_blend_fwd<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, order, vals, mean2d, conic_opacity, color, image,
                                                    final_T, n_contrib);
  return 1;
}

int launch_blend_bwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                     const float *mean2d,
                     const float *conic_opacity, const float *color, const float *final_T,
                     const uint32_t *n_contrib, const float *dL_dimage, float *g2d, cudaStream_t st) {
  k_blend_bwd<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, order, vals, mean2d, conic_opacity, color, final_T,
                                                    n_contrib, dL_dimage, g2d);
  return 1;
}

}  // namespace gs
