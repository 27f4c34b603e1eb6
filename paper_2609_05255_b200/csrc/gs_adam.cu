// Fused Adam update (App. C.1: Adam with one learning rate per column of a parameter tensor; App. C.2:
// fp32 master values with a half-precision copy made for the next iteration).  All tensors of a
// model are updated by ONE launch: a persistent grid walks a common space of 4096-element chunks,
// each thread moving 16-byte vectors.  The kernel is a pure stream - 16 B read and 12 B written per
// element (+ 2 B for the half copy) - so HBM bandwidth bounds it.
#include <cuda_fp16.h>

#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kAdamThreads = 256;
constexpr int kAdamVec = 4;                                    // elements per 16-byte access
constexpr int kAdamUnroll = 4;
constexpr int kAdamChunk = kAdamThreads * kAdamVec * kAdamUnroll;   // 4096 elements

struct AdamTensorDev {
  float *param;
  const float *grad;
  float *m, *v;
  __half *half_copy;
  uint32_t count;            // rows * cols
  uint32_t cols;
  float beta1, beta2, eps;
  float inv_sqrt_c2;         // 1 / sqrt(1 - beta2^step)
  float step_size[GS_ADAM_MAX_COLS];   // lr_c / (1 - beta1^step)
  int num_more;
  const float *more[GS_ADAM_MAX_MORE_GRADS];   // further gradient buffers, summed with grad
};

struct AdamArgs {
  int num_tensors;
  uint32_t chunk_start[GS_ADAM_MAX_TENSORS + 1];   // prefix sum of the tensors' chunk counts
  AdamTensorDev t[GS_ADAM_MAX_TENSORS];
};

__device__ __forceinline__ void adam_element(float &p, float g, float &m, float &v, float step_size, float beta1,
                                             float beta2, float eps, float inv_sqrt_c2) {
  m = fmaf(beta1, m, (1.f - beta1) * g);
  v = fmaf(beta2, v, (1.f - beta2) * g * g);
  const float denom = fmaf(sqrtf(v), inv_sqrt_c2, eps);
  p = fmaf(-step_size, m / denom, p);
}

__global__ void __launch_bounds__(kAdamThreads) k_adam(const __grid_constant__ AdamArgs a) {
  // the per-column step sizes of the chunk's tensor, in shared memory: the lanes of a warp want
  // different columns, which the constant bank would serve one address at a time
  __shared__ float s_step[GS_ADAM_MAX_COLS];
  const uint32_t total_chunks = a.chunk_start[a.num_tensors];
  for (uint32_t chunk = blockIdx.x; chunk < total_chunks; chunk += gridDim.x) {
    int ti = 0;
    while (ti + 1 < a.num_tensors && chunk >= a.chunk_start[ti + 1]) ++ti;
    const AdamTensorDev &t = a.t[ti];
    __syncthreads();
    if (threadIdx.x < t.cols) s_step[threadIdx.x] = t.step_size[threadIdx.x];
    __syncthreads();
    const uint32_t base = (chunk - a.chunk_start[ti]) * kAdamChunk;
    float4 p[kAdamUnroll], g[kAdamUnroll], m[kAdamUnroll], v[kAdamUnroll];
    uint32_t e[kAdamUnroll];
    bool full[kAdamUnroll];
    // all loads of the chunk first
#pragma unroll
    for (int u = 0; u < kAdamUnroll; ++u) {
      e[u] = base + (u * kAdamThreads + threadIdx.x) * kAdamVec;
      full[u] = e[u] + kAdamVec <= t.count;
      if (full[u]) {
        p[u] = *reinterpret_cast<const float4 *>(t.param + e[u]);
        g[u] = __ldcs(reinterpret_cast<const float4 *>(t.grad + e[u]));
        for (int k = 0; k < t.num_more; ++k) {
          const float4 x = __ldcs(reinterpret_cast<const float4 *>(t.more[k] + e[u]));
          g[u].x += x.x; g[u].y += x.y; g[u].z += x.z; g[u].w += x.w;
        }
        m[u] = *reinterpret_cast<const float4 *>(t.m + e[u]);
        v[u] = *reinterpret_cast<const float4 *>(t.v + e[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kAdamUnroll; ++u) {
      if (full[u]) {
        uint32_t c = e[u] % t.cols;
        float *pp = &p[u].x, *mm = &m[u].x, *vv = &v[u].x;
        const float *gg = &g[u].x;
#pragma unroll
        for (int k = 0; k < kAdamVec; ++k) {
          adam_element(pp[k], gg[k], mm[k], vv[k], s_step[c], t.beta1, t.beta2, t.eps, t.inv_sqrt_c2);
          c = (c + 1 == t.cols) ? 0u : c + 1;
        }
        *reinterpret_cast<float4 *>(t.param + e[u]) = p[u];
        *reinterpret_cast<float4 *>(t.m + e[u]) = m[u];
        *reinterpret_cast<float4 *>(t.v + e[u]) = v[u];
        if (t.half_copy) {
          const __half2 lo = __floats2half2_rn(p[u].x, p[u].y), hi = __floats2half2_rn(p[u].z, p[u].w);
          uint2 packed;
          packed.x = *reinterpret_cast<const uint32_t *>(&lo);
          packed.y = *reinterpret_cast<const uint32_t *>(&hi);
          *reinterpret_cast<uint2 *>(t.half_copy + e[u]) = packed;
        }
      } else if (e[u] < t.count) {   // ragged end of the tensor, element by element
        uint32_t c = e[u] % t.cols;
        for (uint32_t i = e[u]; i < t.count; ++i) {
          float pv = t.param[i], mv = t.m[i], vv = t.v[i], gv = t.grad[i];
          for (int k = 0; k < t.num_more; ++k) gv += t.more[k][i];
          adam_element(pv, gv, mv, vv, s_step[c], t.beta1, t.beta2, t.eps, t.inv_sqrt_c2);
          t.param[i] = pv; t.m[i] = mv; t.v[i] = vv;
          if (t.half_copy) t.half_copy[i] = __float2half_rn(pv);
          c = (c + 1 == t.cols) ? 0u : c + 1;
        }
      }
    }
  }
}

}  // namespace

// Host side of gs_adam_step: validates nothing (the C entry point does), fills the argument block,
// launches.  Returns the number of kernels launched.
int launch_adam(const GsAdamTensor *tensors, int num_tensors, int64_t step, int num_sms, cudaStream_t st) {
  AdamArgs a;
  a.num_tensors = 0;
  a.chunk_start[0] = 0;
  for (int i = 0; i < num_tensors; ++i) {
    const GsAdamTensor &s = tensors[i];
    const uint64_t count = (uint64_t)s.rows * (uint64_t)s.cols;
    if (count == 0) continue;
    AdamTensorDev &d = a.t[a.num_tensors];
    d.param = s.param; d.grad = s.grad; d.m = s.exp_avg; d.v = s.exp_avg_sq;
    d.half_copy = reinterpret_cast<__half *>(s.half_copy);
    d.count = (uint32_t)count; d.cols = (uint32_t)s.cols;
    d.beta1 = s.beta1; d.beta2 = s.beta2; d.eps = s.eps;
    const double c1 = 1.0 - pow((double)s.beta1, (double)step), c2 = 1.0 - pow((double)s.beta2, (double)step);
    d.inv_sqrt_c2 = (float)(1.0 / sqrt(c2));
    for (int c = 0; c < s.cols; ++c) d.step_size[c] = (float)((double)s.lr[c] / c1);
    d.num_more = s.more_grads ? s.num_more_grads : 0;
    for (int k = 0; k < d.num_more; ++k) d.more[k] = s.more_grads[k];
    a.chunk_start[a.num_tensors + 1] = a.chunk_start[a.num_tensors] + (uint32_t)((count + kAdamChunk - 1) / kAdamChunk);
    ++a.num_tensors;
  }
  const uint32_t chunks = a.chunk_start[a.num_tensors];
  if (chunks == 0) return 0;
  const uint32_t wave = (uint32_t)num_sms * 8u;
  k_adam<<<chunks < wave ? chunks : wave, kAdamThreads, 0, st>>>(a);
  return 1;
}

}  // namespace gs
