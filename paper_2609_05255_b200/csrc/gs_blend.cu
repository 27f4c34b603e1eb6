// Per-tile alpha blending, forward and backward.  One CTA of 64 threads per 16x16 tile; every
// thread owns a 2x2 pixel quad (a warp covers 16x8 pixels), so one shared-memory read of a
// Gaussian serves four pixels and, in the backward, four pixels are summed in registers before
// anything crosses lanes.  The tile's depth-ordered instance list is staged through shared memory
// in batches of 128 Gaussians (64 in the backward, which also keeps the batch's gradient sums there).
#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kThreads = 64;
constexpr int kBatch = 128;
constexpr int kBatchBwd = 64;   // the backward keeps ten accumulators per entry and warp in shared memory
constexpr unsigned kFull = 0xffffffffu;
constexpr float kLn2 = 0.6931471805599453f;

// Top-left pixel of this thread's quad.
__device__ __forceinline__ void quad_of(int tile, int gx, int tid, int &px, int &py) {
  const int tx = tile % gx, ty = tile / gx;
  const int warp = tid >> 5, lane = tid & 31;
  px = tx * GS_TILE + 2 * (lane & 7);
  py = ty * GS_TILE + warp * 8 + 2 * (lane >> 3);
}

// Stage one batch entry: (x, y, la, lb) (lc, o) (r, g, b, pmin).  (la, lb, lc) is the Cholesky factor
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
  // alpha >= 1/255 <=> log2 falloff >= pmin = -log2(255 o): the test is taken on the exponent, before the
  // exponential, by the forward, the backward and the pair counter alike
  rgb = make_float4(__ldg(color + 3 * (size_t)g), __ldg(color + 3 * (size_t)g + 1), __ldg(color + 3 * (size_t)g + 2),
                    -__log2f(255.f * q.w));
}

// log2 of the Gaussian falloff at the four pixels of a quad; dx0, dy0 are the offsets of the
// top-left pixel centre from the mean.  Index k = 2 * row + column.  One explicit operation order,
// shared by the forward and the backward so that both take identical skip decisions.
// t1[k] = la dx + lb dy is returned too: the backward needs it for the gradient of the mean.
__device__ __forceinline__ void quad_power(float dx0, float dy0, float la, float lb, float lc, float p[4],
                                           float t1[4], float t2[2]) {
  // packed fp32 pairs (one instruction, two IEEE operations): the bits equal the scalar sequence
  const float2 one = make_float2(1.f, 1.f);
  const float2 d1 = __fadd2_rn(make_float2(dx0, dy0), one);            // (dx1, dy1)
  const float2 a = __fmul2_rn(make_float2(la, la), make_float2(dx0, d1.x));
  const float2 c = __fmul2_rn(make_float2(lc, lc), make_float2(dy0, d1.y));
  const float2 s = __fmul2_rn(c, c);
  const float2 lb2 = make_float2(lb, lb);
  const float2 u = __ffma2_rn(lb2, make_float2(dy0, dy0), a), w = __ffma2_rn(lb2, make_float2(d1.y, d1.y), a);
  const float2 pu = __ffma2_rn(u, u, make_float2(s.x, s.x)), pw = __ffma2_rn(w, w, make_float2(s.y, s.y));
  t2[0] = c.x; t2[1] = c.y;
  t1[0] = u.x; t1[1] = u.y; t1[2] = w.x; t1[3] = w.y;
  p[0] = -pu.x; p[1] = -pu.y; p[2] = -pw.x; p[3] = -pw.y;
}

// alpha of one pixel from its log2 falloff p; false if the pair is skipped (alpha < 1/255, decided as
// p < pmin).  raw = o * exp(power) before the clamp at 0.99.
__device__ __forceinline__ bool alpha_of(float p, float o, float pmin, float &e2, float &raw, float &alpha) {
  if (p < pmin) return false;
  e2 = ex2_approx(p);             // p <= 0 by construction
  raw = __fmul_rn(o, e2);
  alpha = fminf(kAlphaMax, raw);
  return true;
}

// 1.0f where a >= b or either is NaN, else 0.0f; 1.0f where a < b, else 0.0f: masks as numbers, so that what
// depends on them runs as packed multiplies on the FMA pipe instead of selects on the ALU pipe.
__device__ __forceinline__ float set_geu(float a, float b) {
  float d;
  asm("set.geu.f32.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float set_lt(float a, float b) {
  float d;
  asm("set.lt.f32.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float set_le(float a, float b) {
  float d;
  asm("set.le.f32.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.f, -1.f), a); }   // a - b, exact products

// Forward.  The four pixels of a quad travel as two packed pairs, (0, 1) and (2, 3), and the composite of an entry is
// branch-free: "this pixel still composites" (live), "it accepts this entry" (q: alpha >= 1/255, decided on the
// exponent) and "it stops here" (s: T - alpha T < 1e-4) are 0/1 numbers.  A pixel that skips the entry, has stopped
// or stops here enters with weight exactly 0, which leaves its transmittance and colour sums unchanged bit for bit.
__global__ void __launch_bounds__(kThreads) k_blend_fwd(CamDev cam, const uint32_t *__restrict__ ranges,
                                                        const uint32_t *__restrict__ order,
                                                        const uint32_t *__restrict__ vals,
                                                        const float *__restrict__ mean2d,
                                                        const float *__restrict__ conic_opacity,
                                                        const float *__restrict__ color, uint32_t *__restrict__ sorted_tiles,
                                                        float *__restrict__ image,
                                                        float *__restrict__ final_T, uint32_t *__restrict__ n_contrib) {
  dependency_wait();
  __shared__ float4 s_xyab[kBatch];
  __shared__ float2 s_co[kBatch];
  __shared__ float4 s_rgb[kBatch];
  const int tid = threadIdx.x, tile = (int)__ldg(order + blockIdx.x);
  int px, py;
  quad_of(tile, cam.gx, tid, px, py);
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  // the key of every instance of this tile's stretch of the sorted list is the tile id: stores that nothing here waits for
  if (sorted_tiles)
    for (uint32_t p = start + tid; p < end; p += kThreads) sorted_tiles[p] = (uint32_t)tile;
  const float in_x1 = px + 1 < cam.W ? 1.f : 0.f, in_y1 = py + 1 < cam.H ? 1.f : 0.f, in_0 = (px < cam.W && py < cam.H) ? 1.f : 0.f;
  // T is the transmittance while the pixel composites and 0 once it has stopped (then every later weight alpha T is
  // 0 by itself); the value it stopped with is kept in F.  Pixels outside the image start stopped.
  float2 T01 = make_float2(in_0, in_0 * in_x1), T23 = make_float2(in_0 * in_y1, in_0 * in_x1 * in_y1);
  const float2 zero = make_float2(0.f, 0.f), one = make_float2(1.f, 1.f);
  float2 F01 = zero, F23 = zero;
  float2 R01 = zero, R23 = zero, G01 = zero, G23 = zero, B01 = zero, B23 = zero;
  uint32_t last[4] = {0u, 0u, 0u, 0u};      // position + 1 of the last composited entry
  for (uint32_t base = start; base < end; base += kBatch) {
    if (__syncthreads_and((T01.x + T01.y) + (T23.x + T23.y) == 0.f)) break;
#pragma unroll
    for (int h = 0; h < kBatch / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      const uint32_t idx = base + slot;
      if (idx < end) stage_entry(__ldg(vals + idx), mean2d, conic_opacity, color, s_xyab[slot], s_co[slot], s_rgb[slot]);
    }
    __syncthreads();
    const int cnt = (int)min((uint32_t)kBatch, end - base);
    float posf = 0.f;                         // position + 1 inside the batch, as a number (exact)
    float2 last01 = zero, last23 = zero;      // the same of the last entry composited in this batch; 0 = none
    for (int j0 = 0; j0 < cnt; j0 += 8) {
      if (!__any_sync(kFull, (T01.x + T01.y) + (T23.x + T23.y) != 0.f)) break;   // every pixel of the warp has stopped
      const int j1 = min(j0 + 8, cnt);
#pragma unroll 2
      for (int j = j0; j < j1; ++j) {
        const float4 a = s_xyab[j];
        const float2 c = s_co[j];
        float p[4], t1[4], t2[2];
        quad_power(fx - a.x, fy - a.y, a.z, a.w, c.x, p, t1, t2);
        const float4 col = s_rgb[j];
        posf += 1.f;
        const float2 q01 = make_float2(set_geu(p[0], col.w), set_geu(p[1], col.w));
        const float2 q23 = make_float2(set_geu(p[2], col.w), set_geu(p[3], col.w));
        if (!__any_sync(kFull, (q01.x + q01.y) + (q23.x + q23.y) != 0.f)) continue;   // no pixel of the warp takes it
        const float2 o2 = make_float2(c.y, c.y);
        const float2 raw01 = __fmul2_rn(o2, make_float2(ex2_approx(p[0]), ex2_approx(p[1])));
        const float2 raw23 = __fmul2_rn(o2, make_float2(ex2_approx(p[2]), ex2_approx(p[3])));
        const float2 al01 = __fmul2_rn(q01, make_float2(fminf(kAlphaMax, raw01.x), fminf(kAlphaMax, raw01.y)));
        const float2 al23 = __fmul2_rn(q23, make_float2(fminf(kAlphaMax, raw23.x), fminf(kAlphaMax, raw23.y)));
        float2 w01 = __fmul2_rn(al01, T01), w23 = __fmul2_rn(al23, T23);
        // transmittance behind this entry, T (1 - alpha) - in this form, because the backward recovers the
        // transmittances by dividing (1 - alpha) out again and drifts if the forward rounds another expression (ten
        // 2D-gradient values of a 1M-Gaussian view were then off by more than 1e-3 of the sum of their terms); below
        // 1e-4 the pixel stops and the entry is not composited.
        // A live pixel that skips the entry keeps T >= 1e-4 and cannot stop here; a stopped one has T = 0 and
        // "stops" again with nothing to lose.
        const float2 n01 = __fmul2_rn(T01, sub2(one, al01)), n23 = __fmul2_rn(T23, sub2(one, al23));
        const float2 s01 = make_float2(set_lt(n01.x, kTmin), set_lt(n01.y, kTmin));
        const float2 s23 = make_float2(set_lt(n23.x, kTmin), set_lt(n23.y, kTmin));
        const float2 k01 = sub2(one, s01), k23 = sub2(one, s23);
        F01 = __ffma2_rn(s01, T01, F01); F23 = __ffma2_rn(s23, T23, F23);
        w01 = __fmul2_rn(w01, k01); w23 = __fmul2_rn(w23, k23);
        T01 = __fmul2_rn(n01, k01); T23 = __fmul2_rn(n23, k23);
        R01 = __ffma2_rn(make_float2(col.x, col.x), w01, R01); R23 = __ffma2_rn(make_float2(col.x, col.x), w23, R23);
        G01 = __ffma2_rn(make_float2(col.y, col.y), w01, G01); G23 = __ffma2_rn(make_float2(col.y, col.y), w23, G23);
        B01 = __ffma2_rn(make_float2(col.z, col.z), w01, B01); B23 = __ffma2_rn(make_float2(col.z, col.z), w23, B23);
        // last += composited * (position - last)
        const float2 pos2 = make_float2(posf, posf);
        last01 = __ffma2_rn(__fmul2_rn(q01, k01), sub2(pos2, last01), last01);
        last23 = __ffma2_rn(__fmul2_rn(q23, k23), sub2(pos2, last23), last23);
      }
    }
    const uint32_t off = base - start;
    if (last01.x != 0.f) last[0] = off + (uint32_t)last01.x;
    if (last01.y != 0.f) last[1] = off + (uint32_t)last01.y;
    if (last23.x != 0.f) last[2] = off + (uint32_t)last23.x;
    if (last23.y != 0.f) last[3] = off + (uint32_t)last23.y;
  }
  T01 = __fadd2_rn(T01, F01); T23 = __fadd2_rn(T23, F23);    // one of the two is 0
  const float T[4] = {T01.x, T01.y, T23.x, T23.y};
  const float Cr[4] = {R01.x, R01.y, R23.x, R23.y}, Cg[4] = {G01.x, G01.y, G23.x, G23.y}, Cb[4] = {B01.x, B01.y, B23.x, B23.y};
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

__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
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
// "final pixel - prefix" cancels badly for deep entries).  Only its product with the pixel's
// upstream gradient is needed, so one scalar per pixel carries it.
//
// What a pixel sends to a Gaussian's conic and mean is linear in dp = dL/d(power) times
// (1, dx, dy, dx^2, dx dy, dy^2).  The threads therefore sum the six moments of dp in tile-local
// pixel coordinates (half-integers up to 7.5, so the products are exact), a quad of pixels at a
// time, and the moments are shifted to the Gaussian's own centre once per (tile, Gaussian) when
// the batch leaves shared memory.  The opacity gradient needs no sum of its own: alpha = o exp(power)
// where it is not clamped, so dL/do = (sum of dp) / o, the zeroth moment.  Nine values per entry cross
// the warp: the six moments and the colour gradient (warp_reduce9); each warp owns its own copy of the
// batch's accumulators, so no shared-memory atomics are needed; the sums leave with one global
// atomic per value.
// g2d row: (d colour r, g, b, d opacity) (d conic A, B, C, d mean u) (d mean v, -, -, -).
__global__ void __launch_bounds__(kThreads, 16) k_blend_bwd(CamDev cam, const uint32_t *__restrict__ ranges,
                                                        const uint32_t *__restrict__ order,
                                                        const uint32_t *__restrict__ vals,
                                                        const float *__restrict__ mean2d,
                                                        const float *__restrict__ conic_opacity,
                                                        const float *__restrict__ color,
                                                        const float *__restrict__ final_T,
                                                        const uint32_t *__restrict__ n_contrib,
                                                        const float *__restrict__ dL_dimage, float *__restrict__ g2d) {
  __shared__ float4 s_xyab[kBatchBwd];
  __shared__ float2 s_co[kBatchBwd];
  __shared__ float4 s_rgb[kBatchBwd];
  __shared__ uint32_t s_gid[kBatchBwd];
  __shared__ float s_acc[kThreads / 32][kBatchBwd][9];
  __shared__ uint32_t s_max[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, tile = (int)__ldg(order + blockIdx.x);
  int px, py;
  quad_of(tile, cam.gx, tid, px, py);
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  // tile-local coordinates of the quad's pixel centres, origin at the middle of the tile
  const float ox_tile = (float)((tile % cam.gx) * GS_TILE + GS_TILE / 2), oy_tile = (float)((tile / cam.gx) * GS_TILE + GS_TILE / 2);
  const float X0 = fx - ox_tile, X1 = X0 + 1.f, Y0 = fy - oy_tile, Y1 = Y0 + 1.f;
  const float XX0 = X0 * X0, XX1 = X1 * X1, YY0 = Y0 * Y0, YY1 = Y1 * Y1;
  const uint32_t start = __ldg(ranges + 2 * tile), end = __ldg(ranges + 2 * tile + 1);
  const size_t plane = (size_t)cam.W * cam.H;
  uint32_t nc[4];
  float T[4], Gr[4], Gg[4], Gb[4], GS[4];
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
    GS[k] = T[k] * fmaf(Gb[k], cam.bg[2], fmaf(Gg[k], cam.bg[1], Gr[k] * cam.bg[0]));   // G . (light from behind)
    wmax = max(wmax, nc[k]);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) wmax = max(wmax, __shfl_xor_sync(kFull, wmax, s));
  if (lane == 0) s_max[warp] = wmax;
  __syncthreads();
  const uint32_t maxc = max(s_max[0], s_max[1]);
  if (maxc == 0 || start + maxc > end) return;   // nothing composited in this tile
  // value that this lane holds after the reduction (lanes 0, 4, .., 28: one of 0..7; lane 1 stores value 8)
  const int my_value = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
  const int nbatches = (int)((maxc + kBatchBwd - 1) / kBatchBwd);
  // pixels (0, 1) and (2, 3) as packed pairs; nGS carries minus G . (light from behind)
  float2 T01 = make_float2(T[0], T[1]), T23 = make_float2(T[2], T[3]);
  float2 nGS01 = make_float2(-GS[0], -GS[1]), nGS23 = make_float2(-GS[2], -GS[3]);
  const float2 Gr01 = make_float2(Gr[0], Gr[1]), Gr23 = make_float2(Gr[2], Gr[3]);
  const float2 Gg01 = make_float2(Gg[0], Gg[1]), Gg23 = make_float2(Gg[2], Gg[3]);
  const float2 Gb01 = make_float2(Gb[0], Gb[1]), Gb23 = make_float2(Gb[2], Gb[3]);
  for (int b = nbatches - 1; b >= 0; --b) {
    __syncthreads();
    const uint32_t first = (uint32_t)b * kBatchBwd;
    const int cnt = (int)min((uint32_t)kBatchBwd, maxc - first);
#pragma unroll
    for (int h = 0; h < kBatchBwd / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      if (slot < cnt) {
        const uint32_t g = __ldg(vals + start + first + slot);
        s_gid[slot] = g;
        stage_entry(g, mean2d, conic_opacity, color, s_xyab[slot], s_co[slot], s_rgb[slot]);
      }
#pragma unroll
      for (int k = 0; k < 9; ++k) s_acc[0][slot][k] = s_acc[1][slot][k] = 0.f;
    }
    __syncthreads();
    const int jtop = (int)min((uint32_t)cnt, wmax > first ? wmax - first : 0u);
    // positions of this batch that each pixel composited: j < lim[k] (as numbers: the comparisons below make 0 / 1 masks)
    float limf[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) limf[k] = nc[k] > first ? (float)min(nc[k] - first, (uint32_t)kBatchBwd) : 0.f;
    float jf = (float)jtop;
    for (int j = jtop - 1; j >= 0; --j) {
      const float4 a = s_xyab[j];
      const float2 c = s_co[j];
      float p[4], t1[4], t2[2];
      quad_power(fx - a.x, fy - a.y, a.z, a.w, c.x, p, t1, t2);
      const float4 col = s_rgb[j];
      jf -= 1.f;
      // q: the pixel composited this entry (it lies inside the pixel's walk and alpha >= 1/255), as 0 / 1
      const float2 q01 = __fmul2_rn(make_float2(set_geu(p[0], col.w), set_geu(p[1], col.w)), make_float2(set_lt(jf, limf[0]), set_lt(jf, limf[1])));
      const float2 q23 = __fmul2_rn(make_float2(set_geu(p[2], col.w), set_geu(p[3], col.w)), make_float2(set_lt(jf, limf[2]), set_lt(jf, limf[3])));
      if (!__any_sync(kFull, (q01.x + q01.y) + (q23.x + q23.y) != 0.f)) continue;
      // Branch-free from here, two packed pixel pairs: a pixel that did not composite this entry enters with
      // alpha = 0, for which the reciprocal is 1, every product below is 0 and its carried state is unchanged.
      const float2 o2 = make_float2(c.y, c.y), one = make_float2(1.f, 1.f), mone = make_float2(-1.f, -1.f);
      const float2 raw01 = __fmul2_rn(o2, make_float2(ex2_approx(p[0]), ex2_approx(p[1])));
      const float2 raw23 = __fmul2_rn(o2, make_float2(ex2_approx(p[2]), ex2_approx(p[3])));
      const float2 al01 = __fmul2_rn(q01, make_float2(fminf(kAlphaMax, raw01.x), fminf(kAlphaMax, raw01.y)));
      const float2 al23 = __fmul2_rn(q23, make_float2(fminf(kAlphaMax, raw23.x), fminf(kAlphaMax, raw23.y)));
      const float2 d01 = __ffma2_rn(al01, mone, one), d23 = __ffma2_rn(al23, mone, one);
      const float2 inv01 = make_float2(rcp_approx(d01.x), rcp_approx(d01.y)), inv23 = make_float2(rcp_approx(d23.x), rcp_approx(d23.y));
      const float2 Tb01 = __fmul2_rn(T01, inv01), Tb23 = __fmul2_rn(T23, inv23);     // transmittance in front of this entry
      const float2 w01 = __fmul2_rn(al01, Tb01), w23 = __fmul2_rn(al23, Tb23);
      float v[9];
      {
        const float2 r = __ffma2_rn(w01, Gr01, __fmul2_rn(w23, Gr23)), g = __ffma2_rn(w01, Gg01, __fmul2_rn(w23, Gg23));
        const float2 bl = __ffma2_rn(w01, Gb01, __fmul2_rn(w23, Gb23));
        v[6] = r.x + r.y; v[7] = g.x + g.y; v[8] = bl.x + bl.y;
      }
      // d pixel / d alpha = T c - S / (1 - alpha), S = everything composited behind this entry
      const float2 cx = make_float2(col.x, col.x), cy = make_float2(col.y, col.y), cz = make_float2(col.z, col.z);
      const float2 gc01 = __ffma2_rn(Gb01, cz, __ffma2_rn(Gg01, cy, __fmul2_rn(Gr01, cx)));
      const float2 gc23 = __ffma2_rn(Gb23, cz, __ffma2_rn(Gg23, cy, __fmul2_rn(Gr23, cx)));
      const float2 da01 = __fmul2_rn(__ffma2_rn(T01, gc01, nGS01), inv01), da23 = __fmul2_rn(__ffma2_rn(T23, gc23, nGS23), inv23);
      // clamped at 0.99: alpha does not depend on opacity and power there (mask 0)
      const float2 e01 = __fmul2_rn(__fmul2_rn(al01, da01), make_float2(set_le(raw01.x, kAlphaMax), set_le(raw01.y, kAlphaMax)));
      const float2 e23 = __fmul2_rn(__fmul2_rn(al23, da23), make_float2(set_le(raw23.x, kAlphaMax), set_le(raw23.y, kAlphaMax)));
      const float dp0 = e01.x, dp1 = e01.y, dp2 = e23.x, dp3 = e23.y;
      nGS01 = __ffma2_rn(make_float2(-w01.x, -w01.y), gc01, nGS01);
      nGS23 = __ffma2_rn(make_float2(-w23.x, -w23.y), gc23, nGS23);
      T01 = Tb01; T23 = Tb23;
      {
        const float sL = dp0 + dp2, sR = dp1 + dp3, sT = dp0 + dp1, sB = dp2 + dp3;
        v[0] = sL + sR;
        v[1] = fmaf(X0, sL, X1 * sR);
        v[2] = fmaf(Y0, sT, Y1 * sB);
        v[3] = fmaf(XX0, sL, XX1 * sR);
        v[4] = fmaf(X0, fmaf(Y0, dp0, Y1 * dp2), X1 * fmaf(Y0, dp1, Y1 * dp3));
        v[5] = fmaf(YY0, sT, YY1 * sB);
        float mine, ninth;
        warp_reduce9(v, lane, mine, ninth);
        if ((lane & 3) == 0) s_acc[warp][j][my_value] = mine;
        if (lane == 1) s_acc[warp][j][8] = ninth;
      }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < kBatchBwd / kThreads; ++h) {
      const int slot = tid + h * kThreads;
      if (slot < cnt) {
        float M[9];
        bool touched = false;
#pragma unroll
        for (int k = 0; k < 9; ++k) {
          M[k] = s_acc[0][slot][k] + s_acc[1][slot][k];
          touched = touched || (M[k] != 0.f);
        }
        if (touched) {
          // moments about the Gaussian's centre from the tile-local ones: d = (X + ox, Y + oy)
          const float4 a = s_xyab[slot];
          const float lc = s_co[slot].x, o = s_co[slot].y;
          const float ox = ox_tile - a.x, oy = oy_tile - a.y;
          const float sx = fmaf(ox, M[0], M[1]), sy = fmaf(oy, M[0], M[2]);
          const float sxx = fmaf(ox, M[1] + sx, M[3]);
          const float sxy = fmaf(oy, sx, fmaf(ox, M[2], M[4]));
          const float syy = fmaf(oy, M[2] + sy, M[5]);
          // the staged factor is the conic's Cholesky factor times sqrt(0.5 log2 e)
          const float A = 2.f * kLn2 * a.z * a.z, B = 2.f * kLn2 * a.z * a.w, C = 2.f * kLn2 * fmaf(a.w, a.w, lc * lc);
          float *dst = g2d + (size_t)s_gid[slot] * 12;
          atomicAdd(dst + 0, M[6]); atomicAdd(dst + 1, M[7]); atomicAdd(dst + 2, M[8]); atomicAdd(dst + 3, __fdividef(M[0], o));
          atomicAdd(dst + 4, -0.5f * sxx); atomicAdd(dst + 5, -sxy); atomicAdd(dst + 6, -0.5f * syy);
          atomicAdd(dst + 7, fmaf(A, sx, B * sy)); atomicAdd(dst + 8, fmaf(B, sx, C * sy));
        }
      }
    }
  }
}

// Measurement only: replay the forward's decisions and count, over all pixels, the list entries
// evaluated (until each pixel stopped) and the pairs composited; and per warp (16 x 8 pixels) the
// entries it walked and those among them that none of its live pixels accepted.
// counts[0] += evaluated, counts[1] += composited, counts[2] += (warp, entry) steps, counts[3] += steps without a taker.
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
  unsigned long long evaluated = 0, composited = 0, steps = 0, idle = 0;
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
    for (int j = 0; j < cnt; ++j) {
      if (!__any_sync(kFull, live != 0)) break;
      const float4 a = s_xyab[j];
      const float2 c = s_co[j];
      float p[4], t1[4], t2[2];
      quad_power(fx - a.x, fy - a.y, a.z, a.w, c.x, p, t1, t2);
      const float4 col = s_rgb[j];
      evaluated += __popc(live);
      bool taken = false;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float e2, raw, alpha;
        if (!((live >> k) & 1u) || !alpha_of(p[k], c.y, col.w, e2, raw, alpha)) continue;
        taken = true;
        const float Tn = __fadd_rn(T[k], -__fmul_rn(alpha, T[k]));
        if (Tn < kTmin) { live &= ~(1u << k); continue; }
        T[k] = Tn;
        ++composited;
      }
      ++steps;
      if (!__any_sync(kFull, taken)) ++idle;
    }
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    evaluated += __shfl_xor_sync(kFull, evaluated, s);
    composited += __shfl_xor_sync(kFull, composited, s);
  }
  if ((tid & 31) == 0) {
    atomicAdd(counts, evaluated); atomicAdd(counts + 1, composited);
    atomicAdd(counts + 2, steps); atomicAdd(counts + 3, idle);     // warp-uniform: one lane speaks for the warp
  }
}

}  // namespace

int launch_blend_count(const CamDev &cam, const uint32_t *ranges, const uint32_t *vals, const float *mean2d,
                       const float *conic_opacity, const float *color, unsigned long long *counts, cudaStream_t st) {
  k_blend_count<<<cam.gx * cam.gy, kThreads, 0, st>>>(cam, ranges, vals, mean2d, conic_opacity, color, counts);
  return 1;
}

int launch_blend_fwd(const CamDev &cam, const uint32_t *ranges, const uint32_t *order, const uint32_t *vals,
                     const float *mean2d,
                     const float *conic_opacity, const float *color, uint32_t *sorted_tiles, float *image, float *final_T,
                     uint32_t *n_contrib, cudaStream_t st) {
  launch_chained(k_blend_fwd, cam.gx * cam.gy, kThreads, 0, st, cam, ranges, order, vals, mean2d, conic_opacity, color, sorted_tiles, image,
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
