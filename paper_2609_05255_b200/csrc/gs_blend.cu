// Per-tile alpha blending, forward and backward.  One CTA per 16x16 tile, one thread per pixel
// (each warp owns an 8x4 pixel patch); the tile's depth-ordered instance list is staged through
// shared memory in batches of 256 Gaussians.
#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 256;
constexpr unsigned kFull = 0xffffffffu;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void pixel_of(int tile, int gx, int tid, int &px, int &py) {
  const int tx = tile % gx, ty = tile / gx;
  const int warp = tid >> 5, lane = tid & 31;
  px = tx * GS_TILE + (warp & 1) * 8 + (lane & 7);
  py = ty * GS_TILE + (warp >> 1) * 4 + (lane >> 3);
}

// Stage one batch entry: (x, y, qa, qb) (qc, o) (r, g, b, -) with the conic pre-scaled so that
// exp(power) = 2^(qa dx^2 + qb dx dy + qc dy^2).
__device__ __forceinline__ void stage_entry(uint32_t g, const float *mean2d, const float *conic_opacity,
                                            const float *color, float4 &xyab, float2 &co, float4 &rgb) {
  const float2 m = __ldg(reinterpret_cast<const float2 *>(mean2d) + g);
  const float4 q = __ldg(reinterpret_cast<const float4 *>(conic_opacity) + g);
  xyab = make_float4(m.x, m.y, -0.5f * kLog2e * q.x, -kLog2e * q.y);
  co = make_float2(-0.5f * kLog2e * q.z, q.w);
  rgb = make_float4(__ldg(color + 3 * (size_t)g), __ldg(color + 3 * (size_t)g + 1), __ldg(color + 3 * (size_t)g + 2), 0.f);
}

__global__ void __launch_bounds__(kThreads) k_blend_fwd(CamDev cam, const uint32_t *__restrict__ ranges,
                                                        const uint32_t *__restrict__ vals,
                                                        const float *__restrict__ mean2d,
                                                        const float *__restrict__ conic_opacity,
                                                        const float *__restrict__ color, float *__restrict__ image,
                                                        float *__restrict__ final_T, uint32_t *__restrict__ n_contrib) {
  __shared__ float4 s_xyab[kBatch];
  __shared__ float2 s_co[kBatch];
  __shared__ float4 s_rgb[kBatch];
  const int tid = threadIdx.x, tile = blockIdx.x;
  int px, py;
  pixel_of(tile, cam.gx, tid, px, py);
  const bool inside = px < cam.W && py < cam.H;
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  float T = 1.f, Cr = 0.f, Cg = 0.f, Cb = 0.f;
  uint32_t last = 0;
  bool done = !inside;
  for (uint32_t base = start; base < end; base += kBatch) {
    if (__syncthreads_and(done)) break;
    const uint32_t idx = base + tid;
    if (idx < end) stage_entry(__ldg(vals + idx), mean2d, conic_opacity, color, s_xyab[tid], s_co[tid], s_rgb[tid]);
    __syncthreads();
    const int cnt = (int)min((uint32_t)kBatch, end - base);
    if (!done) {
      for (int j = 0; j < cnt; ++j) {
        const float4 a = s_xyab[j];
        const float2 c = s_co[j];
        float e2, alpha;
        if (!eval_alpha(fx - a.x, fy - a.y, a.z, a.w, c.x, c.y, e2, alpha)) continue;
        const float Tn = __fmul_rn(T, 1.f - alpha);
        if (Tn < kTmin) { done = true; break; }
        const float w = __fmul_rn(alpha, T);
        const float4 col = s_rgb[j];
        Cr = fmaf(col.x, w, Cr); Cg = fmaf(col.y, w, Cg); Cb = fmaf(col.z, w, Cb);
        T = Tn;
        last = base - start + (uint32_t)j + 1u;
      }
    }
  }
  if (inside) {
    const size_t pix = (size_t)py * cam.W + px, plane = (size_t)cam.W * cam.H;
    image[pix] = fmaf(T, cam.bg[0], Cr);
    image[plane + pix] = fmaf(T, cam.bg[1], Cg);
    image[2 * plane + pix] = fmaf(T, cam.bg[2], Cb);
    final_T[pix] = T;
    n_contrib[pix] = last;
  }
}

// Backward: walk each pixel's composited entries back to front.  The transmittance in front of
// an entry is recovered by dividing out (1 - alpha); the light arriving from behind it is summed
// up on the way (both stay relatively accurate: a front-to-back replay that forms that light as
// "final pixel - prefix" cancels badly for deep entries).  The nine per-Gaussian partial
// derivatives are aggregated over the tile: warp shuffles -> shared-memory accumulators -> one
// global atomic per value.
// g2d row: (d colour r, g, b, d opacity) (d conic A, B, C, d mean u) (d mean v, -, -, -).
__global__ void __launch_bounds__(kThreads) k_blend_bwd(CamDev cam, const uint32_t *__restrict__ ranges,
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
  __shared__ uint32_t s_max;
  const int tid = threadIdx.x, lane = tid & 31, tile = blockIdx.x;
  int px, py;
  pixel_of(tile, cam.gx, tid, px, py);
  const bool inside = px < cam.W && py < cam.H;
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  const size_t pix = (size_t)py * cam.W + px, plane = (size_t)cam.W * cam.H;
  uint32_t nc = 0;
  float Gr = 0.f, Gg = 0.f, Gb = 0.f, Tfin = 1.f;
  if (inside) {
    nc = __ldg(n_contrib + pix);
    Gr = __ldg(dL_dimage + pix); Gg = __ldg(dL_dimage + plane + pix); Gb = __ldg(dL_dimage + 2 * plane + pix);
    Tfin = __ldg(final_T + pix);
  }
  if (tid == 0) s_max = 0;
  __syncthreads();
  uint32_t wmax = nc;
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) wmax = max(wmax, __shfl_xor_sync(kFull, wmax, s));
  if (lane == 0 && wmax) atomicMax(&s_max, wmax);
  __syncthreads();
  const uint32_t maxc = s_max;
  if (maxc == 0 || start + maxc > end) return;   // nothing composited in this tile
  float T = Tfin;                                          // transmittance behind the current entry
  float Sr = Tfin * cam.bg[0], Sg = Tfin * cam.bg[1], Sb = Tfin * cam.bg[2];   // light from behind it
  const int nbatches = (int)((maxc + kBatch - 1) / kBatch);
  for (int b = nbatches - 1; b >= 0; --b) {
    __syncthreads();
    const uint32_t first = (uint32_t)b * kBatch;
    const int cnt = (int)min((uint32_t)kBatch, maxc - first);
    if (tid < cnt) {
      const uint32_t g = __ldg(vals + start + first + tid);
      s_gid[tid] = g;
      stage_entry(g, mean2d, conic_opacity, color, s_xyab[tid], s_co[tid], s_rgb[tid]);
    }
#pragma unroll
    for (int k = 0; k < 9; ++k) s_acc[tid][k] = 0.f;
    __syncthreads();
    const int jtop = (int)min((uint32_t)cnt, wmax > first ? wmax - first : 0u);
    for (int j = jtop - 1; j >= 0; --j) {
      const uint32_t pos = first + (uint32_t)j;
      bool ok = pos < nc;
      float v[9];
#pragma unroll
      for (int k = 0; k < 9; ++k) v[k] = 0.f;
      if (ok) {
        const float4 a = s_xyab[j];
        const float2 c = s_co[j];
        const float dx = fx - a.x, dy = fy - a.y;
        float e2, alpha;
        ok = eval_alpha(dx, dy, a.z, a.w, c.x, c.y, e2, alpha);
        if (ok) {
          const float4 col = s_rgb[j];
          const float inv = __frcp_rn(1.f - alpha);
          const float Tb = T * inv;                 // transmittance in front of this entry
          const float w = alpha * Tb;
          v[0] = w * Gr; v[1] = w * Gg; v[2] = w * Gb;
          // d pixel / d alpha = T c - S / (1 - alpha), S = everything composited behind this entry
          const float dalpha = Gr * (Tb * col.x - Sr * inv) + Gg * (Tb * col.y - Sg * inv) + Gb * (Tb * col.z - Sb * inv);
          if (c.y * e2 <= kAlphaMax) {              // not clamped: alpha depends on o and power
            v[3] = e2 * dalpha;
            const float dp = alpha * dalpha;
            const float dp2 = dp * kLn2;            // the staged conic carries a factor log2(e)
            v[4] = -0.5f * dx * dx * dp;
            v[5] = -dx * dy * dp;
            v[6] = -0.5f * dy * dy * dp;
            v[7] = -dp2 * (2.f * a.z * dx + a.w * dy);
            v[8] = -dp2 * (a.w * dx + 2.f * c.x * dy);
          }
          Sr = fmaf(col.x, w, Sr); Sg = fmaf(col.y, w, Sg); Sb = fmaf(col.z, w, Sb);
          T = Tb;
        }
      }
      if (__any_sync(kFull, ok)) {
#pragma unroll
        for (int k = 0; k < 9; ++k) {
#pragma unroll
          for (int s = 16; s > 0; s >>= 1) v[k] += __shfl_xor_sync(kFull, v[k], s);
        }
        if (lane == 0) {
#pragma unroll
          for (int k = 0; k < 9; ++k) atomicAdd(&s_acc[j][k], v[k]);
        }
      }
    }
    __syncthreads();
    if (tid < cnt) {
      float *dst = g2d + (size_t)s_gid[tid] * 12;
      bool any = false;
#pragma unroll
      for (int k = 0; k < 9; ++k) any = any || (s_acc[tid][k] != 0.f);
      if (any) {
#pragma unroll
        for (int k = 0; k < 9; ++k) atomicAdd(dst + k, s_acc[tid][k]);
      }
    }
  }
}

}  // namespace

int launch_blend_fwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *vals, const float *mean2d,
                      const float *conic_opacity, const float *color, float *image, float *final_T,
                      uint32_t *n_contrib, cudaStream_t st) {
  k_blend_fwd<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, vals, mean2d, conic_opacity, color, image,
                                                    final_T, n_contrib);
  return 1;
}

int launch_blend_bwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *vals, const float *mean2d,
                      const float *conic_opacity, const float *color, const float *final_T,
                      const uint32_t *n_contrib, const float *dL_dimage, float *g2d, cudaStream_t st) {
  k_blend_bwd<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, vals, mean2d, conic_opacity, color, final_T,
                                                    n_contrib, dL_dimage, g2d);
  return 1;
}

}  // namespace gs
