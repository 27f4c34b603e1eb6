// CPU oracle for the differentiable Gaussian-splatting step with fused view-dependent
// appearance.  TEST INFRASTRUCTURE ONLY: it is imported by tests/, by the smoke check and by
// the benchmark's cpu_baseline leg, never by the product path, and it shares no code with
// the CUDA kernels.
//
// Plain, slow, double precision.  Every function takes HOST pointers.  Float parameters are
// passed as double (fp32 / fp16 inputs are widened exactly by the caller), so that central
// finite differences can be taken on the same code.  OpenMP "parallel for" over Gaussians
// and tiles is the only parallelism; every reduction is done in a fixed order.
//
// What each part follows:
//   * preprocess (projection of a 3D Gaussian to the image plane, 16x16 tiles): Sec. 3.1
//     "Appearance Modelling in Gaussian Splatting" (preprocess kernel) with the standard
//     EWA-splatting formulation the paper builds on.
//   * SH colour: Eq. 1 in the common-interface form of Eq. 2 (Y0 folded into c0,
//     phi(x) = ReLU(x + 0.5)).
//   * neural colour: Eq. 5 (input), Eq. 6 (frequency encoding, k = 1), Eq. 7 (tanh residual);
//     32 -> 16 ReLU -> 16 ReLU -> 3, no biases (Sec. 4); progressive schedule (Sec. 4 and
//     App. A "Neural": inactive inputs are zero, residual disabled at degree 0).
//   * blend: Sec. 3.1 (blend kernel: per-tile front-to-back alpha compositing in depth order).
//   * backward: analytic derivatives of the above; directional colour gradient reaches the
//     mean (Sec. 4 "CUDA Implementation").
//
// Pins: tests/test_oracle_*.py (closed forms, invariants, brute force, finite differences).
// No function here is "parity unpinned".

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

constexpr double kPi = 3.14159265358979323846;
constexpr double kAlphaMin = 1.0 / 255.0;
constexpr double kAlphaMax = 0.99;
constexpr double kTmin = 1e-4;
constexpr double kDilation = 0.3;
constexpr int kTile = 16;

struct Cam {
  int W, H;
  double fx, fy, cx, cy;
  double R[9], t[3];
  double near_plane, far_plane;
  double bg[3];
};

Cam read_cam(const double* c) {
  Cam k;
  k.W = (int)c[0]; k.H = (int)c[1];
  k.fx = c[2]; k.fy = c[3]; k.cx = c[4]; k.cy = c[5];
  for (int r = 0; r < 3; ++r) {
    for (int j = 0; j < 3; ++j) k.R[3 * r + j] = c[6 + 4 * r + j];
    k.t[r] = c[6 + 4 * r + 3];
  }
  k.near_plane = c[18]; k.far_plane = c[19];
  k.bg[0] = c[20]; k.bg[1] = c[21]; k.bg[2] = c[22];
  return k;
}

// Rotation matrix of a UNIT quaternion (r, x, y, z), row-major.
void quat_to_rot(const double q[4], double R[9]) {
  const double r = q[0], x = q[1], y = q[2], z = q[3];
  R[0] = 1 - 2 * (y * y + z * z); R[1] = 2 * (x * y - r * z);     R[2] = 2 * (x * z + r * y);
  R[3] = 2 * (x * y + r * z);     R[4] = 1 - 2 * (x * x + z * z); R[5] = 2 * (y * z - r * x);
  R[6] = 2 * (x * z - r * y);     R[7] = 2 * (y * z + r * x);     R[8] = 1 - 2 * (x * x + y * y);
}

// Real orthonormal SH basis of degrees 0..3 (order m = -l..l) and the R^3 gradient of each
// polynomial.
void sh_basis(const double d[3], double Y[16]) {
  const double x = d[0], y = d[1], z = d[2];
  const double k1 = std::sqrt(3.0 / (4.0 * kPi));
  const double k2a = 0.5 * std::sqrt(15.0 / kPi), k2b = 0.25 * std::sqrt(5.0 / kPi),
               k2c = 0.25 * std::sqrt(15.0 / kPi);
  const double k3a = 0.25 * std::sqrt(35.0 / (2.0 * kPi)), k3b = 0.5 * std::sqrt(105.0 / kPi),
               k3c = 0.25 * std::sqrt(21.0 / (2.0 * kPi)), k3d = 0.25 * std::sqrt(7.0 / kPi),
               k3e = 0.25 * std::sqrt(105.0 / kPi);
  Y[0] = 0.5 * std::sqrt(1.0 / kPi);
  Y[1] = -k1 * y; Y[2] = k1 * z; Y[3] = -k1 * x;
  Y[4] = k2a * x * y; Y[5] = -k2a * y * z; Y[6] = k2b * (2 * z * z - x * x - y * y);
  Y[7] = -k2a * x * z; Y[8] = k2c * (x * x - y * y);
  Y[9] = -k3a * y * (3 * x * x - y * y);
  Y[10] = k3b * x * y * z;
  Y[11] = -k3c * y * (4 * z * z - x * x - y * y);
  Y[12] = k3d * z * (2 * z * z - 3 * x * x - 3 * y * y);
  Y[13] = -k3c * x * (4 * z * z - x * x - y * y);
  Y[14] = k3e * z * (x * x - y * y);
  Y[15] = -k3a * x * (x * x - 3 * y * y);
}

void sh_basis_grad(const double d[3], double G[16][3]) {
  const double x = d[0], y = d[1], z = d[2];
  const double k1 = std::sqrt(3.0 / (4.0 * kPi));
  const double k2a = 0.5 * std::sqrt(15.0 / kPi), k2b = 0.25 * std::sqrt(5.0 / kPi),
               k2c = 0.25 * std::sqrt(15.0 / kPi);
  const double k3a = 0.25 * std::sqrt(35.0 / (2.0 * kPi)), k3b = 0.5 * std::sqrt(105.0 / kPi),
               k3c = 0.25 * std::sqrt(21.0 / (2.0 * kPi)), k3d = 0.25 * std::sqrt(7.0 / kPi),
               k3e = 0.25 * std::sqrt(105.0 / kPi);
  auto set = [&](int k, double a, double b, double c) { G[k][0] = a; G[k][1] = b; G[k][2] = c; };
  set(0, 0, 0, 0);
  set(1, 0, -k1, 0); set(2, 0, 0, k1); set(3, -k1, 0, 0);
  set(4, k2a * y, k2a * x, 0);
  set(5, 0, -k2a * z, -k2a * y);
  set(6, -2 * k2b * x, -2 * k2b * y, 4 * k2b * z);
  set(7, -k2a * z, 0, -k2a * x);
  set(8, 2 * k2c * x, -2 * k2c * y, 0);
  set(9, -k3a * 6 * x * y, -k3a * (3 * x * x - 3 * y * y), 0);
  set(10, k3b * y * z, k3b * x * z, k3b * x * y);
  set(11, 2 * k3c * x * y, -k3c * (4 * z * z - x * x - 3 * y * y), -8 * k3c * y * z);
  set(12, -6 * k3d * x * z, -6 * k3d * y * z, k3d * (6 * z * z - 3 * x * x - 3 * y * y));
  set(13, -k3c * (4 * z * z - 3 * x * x - y * y), 2 * k3c * x * y, -8 * k3c * x * z);
  set(14, 2 * k3e * x * z, -2 * k3e * y * z, k3e * (x * x - y * y));
  set(15, -k3a * (3 * x * x - 3 * y * y), 6 * k3a * x * y, 0);
}

inline int num_active(int deg) { return (deg + 1) * (deg + 1); }

// Layer sizes of the shared decoder (Sec. 4).
constexpr int kIn = 32, kHid = 16, kOut = 3, kFeat = 8;
constexpr int kW1 = 0, kW2 = kIn * kHid, kW3 = kIn * kHid + kHid * kHid;
constexpr int kNumW = kIn * kHid + kHid * kHid + kHid * kOut;

struct MlpState {
  double x[kIn], h1[kHid], h2[kHid], y[kOut], A[kOut];
  double kink;   // smallest |pre-activation| of the 32 hidden units: how far the nearest ReLU decision is from flipping
};

// Colour activations of Sec. 3.1, as functions of x = c0 + A(d).  All map 0 to (about) 0.5 with slope
// (about) 1:  0: ReLU(x + 0.5)   1: softplus(x + 0.5), beta = 10   2: sigmoid(4 x)   3: clamp(x + 0.5, 0, 1).
// The derivative at a kink is the one-sided value 0.
double color_act(int act, double x) {
  switch (act) {
    case 1: { const double z = 10.0 * (x + 0.5); return (z > 30 ? z : std::log1p(std::exp(z))) / 10.0; }
    case 2: return 1.0 / (1.0 + std::exp(-4.0 * x));
    case 3: { const double z = x + 0.5; return z < 0 ? 0.0 : (z > 1 ? 1.0 : z); }
    default: { const double z = x + 0.5; return z > 0 ? z : 0.0; }
  }
}
double color_act_grad(int act, double x) {
  switch (act) {
    case 1: return 1.0 / (1.0 + std::exp(-10.0 * (x + 0.5)));
    case 2: { const double y = 1.0 / (1.0 + std::exp(-4.0 * x)); return 4.0 * y * (1.0 - y); }
    case 3: { const double z = x + 0.5; return (z > 0 && z < 1) ? 1.0 : 0.0; }
    default: return (x + 0.5) > 0 ? 1.0 : 0.0;
  }
}

// Spherical Voronoi residual (Eq. 3, App. B "Spherical Voronoi"): kSites sites per Gaussian, seven raw
// parameters each, in the order (a_r, a_g, a_b, s_x, s_y, s_z, t): colour a, unnormalised site direction,
// log-temperature.  s = raw / |raw|, tau = exp(t), rho = |s - d| (chord distance),
//   A(d) = sum_i softmax_i(-tau_i rho_i) a_i.
constexpr int kSites = 7, kSiteP = 7;
struct SvState { double s[kSites][3], tau[kSites], rho[kSites], w[kSites], len[kSites]; };
void sv_forward(const double* site, const double d[3], double A[3], SvState& st) {
  double logit[kSites], mx = -1e300;
  for (int i = 0; i < kSites; ++i) {
    const double* p = site + kSiteP * i;
    st.len[i] = std::sqrt(p[3] * p[3] + p[4] * p[4] + p[5] * p[5]);
    for (int c = 0; c < 3; ++c) st.s[i][c] = p[3 + c] / st.len[i];
    st.tau[i] = std::exp(p[6]);
    const double e[3] = {st.s[i][0] - d[0], st.s[i][1] - d[1], st.s[i][2] - d[2]};
    st.rho[i] = std::sqrt(e[0] * e[0] + e[1] * e[1] + e[2] * e[2]);
    logit[i] = -st.tau[i] * st.rho[i];
    mx = std::max(mx, logit[i]);
  }
  double z = 0;
  for (int i = 0; i < kSites; ++i) { st.w[i] = std::exp(logit[i] - mx); z += st.w[i]; }
  A[0] = A[1] = A[2] = 0;
  for (int i = 0; i < kSites; ++i) {
    st.w[i] /= z;
    for (int c = 0; c < 3; ++c) A[c] += st.w[i] * site[kSiteP * i + c];
  }
}
// gA = dL/dA.  g_site [7,7] (written), g_d[3] (added to).  Where rho = 0 the distance has no gradient.
void sv_backward(const double* site, const double d[3], const double gA[3], const SvState& st, const double A[3],
                 double* g_site, double g_d[3]) {
  const double Ag = A[0] * gA[0] + A[1] * gA[1] + A[2] * gA[2];
  for (int i = 0; i < kSites; ++i) {
    const double* p = site + kSiteP * i;
    double* g = g_site + kSiteP * i;
    for (int c = 0; c < 3; ++c) g[c] = st.w[i] * gA[c];
    const double g_logit = st.w[i] * (p[0] * gA[0] + p[1] * gA[1] + p[2] * gA[2] - Ag);
    g[6] = -st.rho[i] * g_logit * st.tau[i];                 // through tau = exp(t)
    const double g_rho = -st.tau[i] * g_logit;
    double gs[3] = {0, 0, 0};
    if (st.rho[i] > 0)
      for (int c = 0; c < 3; ++c) {
        const double u = (st.s[i][c] - d[c]) / st.rho[i];
        gs[c] = g_rho * u;
        g_d[c] -= g_rho * u;
      }
    const double dot = gs[0] * st.s[i][0] + gs[1] * st.s[i][1] + gs[2] * st.s[i][2];   // through the normalisation
    for (int c = 0; c < 3; ++c) g[3 + c] = (gs[c] - dot * st.s[i][c]) / st.len[i];
  }
}

// Eq. 5-7: x = (Y_0..15(d) masked by the active degree, (sin f_j, cos f_j)_j); two ReLU
// layers; A = tanh(W3 h2).
void mlp_forward(const double* W, const double d[3], const double* f, int deg, MlpState& s) {
  double Y[16];
  sh_basis(d, Y);
  const int na = num_active(deg);
  for (int k = 0; k < 16; ++k) s.x[k] = k < na ? Y[k] : 0.0;
  for (int j = 0; j < kFeat; ++j) {
    s.x[16 + 2 * j] = std::sin(f[j]);
    s.x[17 + 2 * j] = std::cos(f[j]);
  }
  s.kink = 1e300;
  for (int o = 0; o < kHid; ++o) {
    double a = 0;
    for (int i = 0; i < kIn; ++i) a += W[kW1 + o * kIn + i] * s.x[i];
    s.h1[o] = a > 0 ? a : 0;
    s.kink = std::min(s.kink, std::fabs(a));
  }
  for (int o = 0; o < kHid; ++o) {
    double a = 0;
    for (int i = 0; i < kHid; ++i) a += W[kW2 + o * kHid + i] * s.h1[i];
    s.h2[o] = a > 0 ? a : 0;
    s.kink = std::min(s.kink, std::fabs(a));
  }
  for (int o = 0; o < kOut; ++o) {
    double a = 0;
    for (int i = 0; i < kHid; ++i) a += W[kW3 + o * kHid + i] * s.h2[i];
    s.y[o] = a;
    s.A[o] = std::tanh(a);
  }
}

template <class F>
void pixel_rect(F u, F v, F ex, F ey, int W, int H, int r[4], bool& empty) {
  // pixel (i, j) has its centre at (i + 0.5, j + 0.5); keep the centres inside the box
  // [u - ex, u + ex] x [v - ey, v + ey].  One rounding per operation, left to right.
  F lo_x = u - ex;  lo_x = lo_x - (F)0.5;
  F hi_x = u + ex;  hi_x = hi_x - (F)0.5;
  F lo_y = v - ey;  lo_y = lo_y - (F)0.5;
  F hi_y = v + ey;  hi_y = hi_y - (F)0.5;
  double i0 = std::ceil((double)lo_x), i1 = std::floor((double)hi_x);
  double j0 = std::ceil((double)lo_y), j1 = std::floor((double)hi_y);
  empty = !(i0 <= i1 && j0 <= j1) || i1 < 0 || j1 < 0 || i0 > W - 1 || j0 > H - 1;
  if (empty) { r[0] = r[1] = r[2] = r[3] = 0; return; }
  r[0] = (int)std::max(i0, 0.0); r[1] = (int)std::min(i1, (double)(W - 1));
  r[2] = (int)std::max(j0, 0.0); r[3] = (int)std::min(j1, (double)(H - 1));
}

inline void tile_rect(const int px[4], int t[4]) {
  t[0] = px[0] >> 4; t[1] = px[2] >> 4; t[2] = (px[1] >> 4) + 1; t[3] = (px[3] >> 4) + 1;
}

}  // namespace

extern "C" {

int gso_num_mlp_weights() { return kNumW; }

// MAC count of one decoder evaluation; fold = 1 counts only what remains when the 16
// feature columns and the constant degree-0 column of the first layer are pre-multiplied
// per Gaussian (App. B.3, first-layer folding).
int gso_mlp_macs(int fold) { return (fold ? 16 : kIn) * kHid + kHid * kHid + kHid * kOut; }

// Viewer-side evaluation of the neural model (App. C.3, "Neural").  The 16 encoded feature inputs and
// the constant degree-0 input do not depend on the view, so their 17 columns of the first layer are
// folded into 16 pre-activations per Gaussian when the model is exported:
//   pre[o] = W1[o][0] Y_0 + sum_j (W1[o][16+2j] sin f_j + W1[o][17+2j] cos f_j).
// deg >= 1 (with deg = 0 the residual is disabled and nothing is folded).
void gso_neural_fold(int64_t n, const double* features, const double* weights, double* pre) {
  const double d0[3] = {0, 0, 1};
  double Y[16];
  sh_basis(d0, Y);   // Y[0] is the constant
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i)
    for (int o = 0; o < kHid; ++o) {
      double a = weights[kW1 + o * kIn + 0] * Y[0];
      for (int j = 0; j < kFeat; ++j) {
        a += weights[kW1 + o * kIn + 16 + 2 * j] * std::sin(features[kFeat * i + j]);
        a += weights[kW1 + o * kIn + 17 + 2 * j] * std::cos(features[kFeat * i + j]);
      }
      pre[kHid * i + o] = a;
    }
}

// Per frame: only the 15 direction-dependent columns (SH degrees 1..3, masked by the active degree)
// of the first layer remain, 15 (padded to 16) x 16 + 16 x 16 + 16 x 3 = 560 multiply-accumulates:
//   h1 = ReLU(pre + W1[:, 1..15] Y_1..15(d)); h2 = ReLU(W2 h1); A = tanh(W3 h2); c = phi(c0 + A).
// d = (mean - eye) / |mean - eye|.
void gso_neural_prepass(int64_t n, int deg, int act, const double* means, const double* base_color, const double* pre,
                        const double* weights, const double* eye, double* color) {
  const int na = num_active(deg);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    double A[3] = {0, 0, 0};
    if (deg > 0) {
      double d[3] = {means[3 * i] - eye[0], means[3 * i + 1] - eye[1], means[3 * i + 2] - eye[2]};
      const double len = std::sqrt(d[0] * d[0] + d[1] * d[1] + d[2] * d[2]);
      for (int c = 0; c < 3; ++c) d[c] /= len;
      double Y[16], h1[kHid], h2[kHid];
      sh_basis(d, Y);
      for (int o = 0; o < kHid; ++o) {
        double a = pre[kHid * i + o];
        for (int k = 1; k < na; ++k) a += weights[kW1 + o * kIn + k] * Y[k];
        h1[o] = a > 0 ? a : 0;
      }
      for (int o = 0; o < kHid; ++o) {
        double a = 0;
        for (int k = 0; k < kHid; ++k) a += weights[kW2 + o * kHid + k] * h1[k];
        h2[o] = a > 0 ? a : 0;
      }
      for (int o = 0; o < kOut; ++o) {
        double a = 0;
        for (int k = 0; k < kHid; ++k) a += weights[kW3 + o * kHid + k] * h2[k];
        A[o] = std::tanh(a);
      }
    }
    for (int c = 0; c < 3; ++c) {
      color[3 * i + c] = color_act(act, base_color[3 * i + c] + A[c]);
    }
  }
}

// One Adam step on a [rows, cols] parameter tensor with one learning rate per column (App. C.1:
// the optimiser is Adam with the single change that it takes a learning rate per column of a
// parameter tensor).  Plain textbook form, step = 1, 2, ...:
//   m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;
//   theta <- theta - lr_c (m / (1 - b1^step)) / (sqrt(v / (1 - b2^step)) + eps).
void gso_adam_step(int64_t rows, int cols, double* param, const double* grad, double* m, double* v,
                   const double* lr, double beta1, double beta2, double eps, int64_t step) {
  const double c1 = 1.0 - std::pow(beta1, (double)step), c2 = 1.0 - std::pow(beta2, (double)step);
  for (int64_t r = 0; r < rows; ++r)
    for (int c = 0; c < cols; ++c) {
      const int64_t i = r * cols + c;
      const double g = grad[i];
      m[i] = beta1 * m[i] + (1.0 - beta1) * g;
      v[i] = beta2 * v[i] + (1.0 - beta2) * g * g;
      const double mhat = m[i] / c1, vhat = v[i] / c2;
      param[i] -= lr[c] * mhat / (std::sqrt(vhat) + eps);
    }
}

void gso_sh_basis(const double* d, double* Y) { sh_basis(d, Y); }
void gso_sh_basis_grad(const double* d, double* G) {
  double g[16][3];
  sh_basis_grad(d, g);
  std::memcpy(G, g, sizeof(g));
}
void gso_quat_to_rot(const double* q, double* R) {
  const double n = std::sqrt(q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3]);
  const double u[4] = {q[0] / n, q[1] / n, q[2] / n, q[3] / n};
  quat_to_rot(u, R);
}

// ---------------------------------------------------------------------------------------
// Per-Gaussian projection.  Outputs (all [n, .]): mean2d[2], cov2d[3] = (a, b, c) with the
// dilation included, conic[3] = (A, B, C), opacity, extent[2], depth32 (float, the sort key),
// dir[3] (unit, camera centre -> mean), valid (passed every cull except "rect empty"),
// visible (valid and rect non-empty), rect_px[4] = (i_min, i_max, j_min, j_max) in double
// arithmetic.
// ---------------------------------------------------------------------------------------
void gso_preprocess(int64_t n, const double* means, const double* log_scales, const double* quats,
                    const double* opacity_logits, const double* cam_, double* mean2d,
                    double* cov2d, double* conic, double* opacity, double* extent, float* depth32,
                    double* dir, uint8_t* valid, uint8_t* visible, int32_t* rect_px) {
  const Cam cam = read_cam(cam_);
  double oc[3];  // camera centre o_c = -R^T t
  for (int j = 0; j < 3; ++j)
    oc[j] = -(cam.R[0 + j] * cam.t[0] + cam.R[3 + j] * cam.t[1] + cam.R[6 + j] * cam.t[2]);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    valid[i] = 0; visible[i] = 0; depth32[i] = 0.f;
    for (int j = 0; j < 2; ++j) { mean2d[2 * i + j] = 0; extent[2 * i + j] = 0; }
    for (int j = 0; j < 3; ++j) { cov2d[3 * i + j] = 0; conic[3 * i + j] = 0; dir[3 * i + j] = 0; }
    for (int j = 0; j < 4; ++j) rect_px[4 * i + j] = 0;
    opacity[i] = 0;
    const double* mu = means + 3 * i;
    bool finite = std::isfinite(opacity_logits[i]);
    for (int j = 0; j < 3; ++j) finite = finite && std::isfinite(mu[j]) && std::isfinite(log_scales[3 * i + j]);
    for (int j = 0; j < 4; ++j) finite = finite && std::isfinite(quats[4 * i + j]);
    if (!finite) continue;
    // depth key: one fused multiply-add chain in fp32 so that any IEEE machine gets the same bits
    const float z32 = std::fmaf((float)cam.R[8], (float)mu[2],
                      std::fmaf((float)cam.R[7], (float)mu[1],
                      std::fmaf((float)cam.R[6], (float)mu[0], (float)cam.t[2])));
    depth32[i] = z32;
    if (!(z32 >= (float)cam.near_plane) || !(z32 <= (float)cam.far_plane)) continue;
    const double o = 1.0 / (1.0 + std::exp(-opacity_logits[i]));
    if (o < kAlphaMin) continue;
    const double tau = 2.0 * std::log(255.0 * o);
    // covariance Sigma = M M^T, M = R diag(s)
    const double* q = quats + 4 * i;
    const double qn = std::sqrt(q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3]);
    if (!(qn > 0)) continue;
    const double qh[4] = {q[0] / qn, q[1] / qn, q[2] / qn, q[3] / qn};
    double R[9];
    quat_to_rot(qh, R);
    double M[9], S[9];
    for (int r = 0; r < 3; ++r)
      for (int k = 0; k < 3; ++k) M[3 * r + k] = R[3 * r + k] * std::exp(log_scales[3 * i + k]);
    for (int r = 0; r < 3; ++r)
      for (int c = 0; c < 3; ++c) {
        double a = 0;
        for (int k = 0; k < 3; ++k) a += M[3 * r + k] * M[3 * c + k];
        S[3 * r + c] = a;
      }
    double t[3];
    for (int r = 0; r < 3; ++r)
      t[r] = cam.R[3 * r] * mu[0] + cam.R[3 * r + 1] * mu[1] + cam.R[3 * r + 2] * mu[2] + cam.t[r];
    const double u = cam.fx * t[0] / t[2] + cam.cx, v = cam.fy * t[1] / t[2] + cam.cy;
    const double limx = 1.3 * (cam.W / 2.0) / cam.fx, limy = 1.3 * (cam.H / 2.0) / cam.fy;
    const double txc = t[2] * std::min(limx, std::max(-limx, t[0] / t[2]));
    const double tyc = t[2] * std::min(limy, std::max(-limy, t[1] / t[2]));
    const double J[6] = {cam.fx / t[2], 0, -cam.fx * txc / (t[2] * t[2]),
                         0, cam.fy / t[2], -cam.fy * tyc / (t[2] * t[2])};
    double T[6];
    for (int r = 0; r < 2; ++r)
      for (int c = 0; c < 3; ++c)
        T[3 * r + c] = J[3 * r] * cam.R[c] + J[3 * r + 1] * cam.R[3 + c] + J[3 * r + 2] * cam.R[6 + c];
    double TS[6];
    for (int r = 0; r < 2; ++r)
      for (int c = 0; c < 3; ++c)
        TS[3 * r + c] = T[3 * r] * S[c] + T[3 * r + 1] * S[3 + c] + T[3 * r + 2] * S[6 + c];
    const double a = TS[0] * T[0] + TS[1] * T[1] + TS[2] * T[2] + kDilation;
    const double b = TS[0] * T[3] + TS[1] * T[4] + TS[2] * T[5];
    const double c = TS[3] * T[3] + TS[4] * T[4] + TS[5] * T[5] + kDilation;
    const double det = a * c - b * b;
    if (!(det > 0) || !std::isfinite(det)) continue;
    const double ex = std::sqrt(tau * a), ey = std::sqrt(tau * c);
    if (!std::isfinite(u) || !std::isfinite(v) || !std::isfinite(ex) || !std::isfinite(ey)) continue;
    valid[i] = 1;
    mean2d[2 * i] = u; mean2d[2 * i + 1] = v;
    cov2d[3 * i] = a; cov2d[3 * i + 1] = b; cov2d[3 * i + 2] = c;
    conic[3 * i] = c / det; conic[3 * i + 1] = -b / det; conic[3 * i + 2] = a / det;
    opacity[i] = o;
    extent[2 * i] = ex; extent[2 * i + 1] = ey;
    double dv[3] = {mu[0] - oc[0], mu[1] - oc[1], mu[2] - oc[2]};
    const double dn = std::sqrt(dv[0] * dv[0] + dv[1] * dv[1] + dv[2] * dv[2]);
    for (int j = 0; j < 3; ++j) dir[3 * i + j] = dv[j] / dn;
    int r[4]; bool empty;
    pixel_rect<double>(u, v, ex, ey, cam.W, cam.H, r, empty);
    if (empty) continue;
    visible[i] = 1;
    for (int j = 0; j < 4; ++j) rect_px[4 * i + j] = r[j];
  }
}

// ---------------------------------------------------------------------------------------
// Appearance decode, c = max(0, c0 + 0.5 + A(d)) (Eq. 2).  app = 0: SH (Eq. 1), app = 1:
// neural (Eq. 5-7).  `mask` (may be null): rows with mask == 0 are skipped (colour 0).
// sh_rest is [n,15,3]; features [n,8]; weights [816] = W1[16][32], W2[16][16], W3[3][16].
// residual_out (may be null) receives A(d).
// ---------------------------------------------------------------------------------------
void gso_appearance_forward(int64_t n, int app, int deg, int act, const double* base_color,
                            const double* sh_rest, const double* features, const double* weights,
                            const double* dirs, const uint8_t* mask, double* color,
                            double* residual_out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    double A[3] = {0, 0, 0};
    for (int c = 0; c < 3; ++c) color[3 * i + c] = 0;
    if (residual_out) for (int c = 0; c < 3; ++c) residual_out[3 * i + c] = 0;
    if (mask && !mask[i]) continue;
    if (app == 0) {
      double Y[16];
      sh_basis(dirs + 3 * i, Y);
      for (int k = 1; k < num_active(deg); ++k)
        for (int c = 0; c < 3; ++c) A[c] += Y[k] * sh_rest[(i * 15 + (k - 1)) * 3 + c];
    } else if (app == 2) {   // Spherical Voronoi: the sites travel in the sh_rest argument, [n,7,7]
      if (deg > 0) { SvState st; sv_forward(sh_rest + (size_t)i * kSites * kSiteP, dirs + 3 * i, A, st); }
    } else if (deg > 0) {
      MlpState s;
      mlp_forward(weights, dirs + 3 * i, features + kFeat * i, deg, s);
      for (int c = 0; c < 3; ++c) A[c] = s.A[c];
    }
    for (int c = 0; c < 3; ++c) {
      color[3 * i + c] = color_act(act, base_color[3 * i + c] + A[c]);
      if (residual_out) residual_out[3 * i + c] = A[c];
    }
  }
}

// Backward of the decode.  g_color = dL/dc.  Outputs: g_base[n,3], g_sh_rest[n,15,3] or
// g_features[n,8], g_weights[816] (sum over Gaussians in index order), g_dirs[n,3] (gradient
// with respect to the direction as a free R^3 vector).
// Per Gaussian, the smallest |pre-activation| among the decoder's 32 hidden units (infinite where the residual is
// disabled): a row whose margin is within fp32 rounding of zero is one where a single-precision evaluation may take
// the other branch of a ReLU.  The parity tests use it to say WHICH rows may differ, instead of only how many.
void gso_mlp_kink_margin(int64_t n, int deg, const double* features, const double* weights, const double* dirs,
                         double* margin) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    margin[i] = INFINITY;
    if (deg <= 0) continue;
    MlpState s;
    mlp_forward(weights, dirs + 3 * i, features + kFeat * i, deg, s);
    margin[i] = s.kink;
  }
}

void gso_appearance_backward(int64_t n, int app, int deg, int act, const double* base_color,
                             const double* sh_rest, const double* features, const double* weights,
                             const double* dirs, const uint8_t* mask, const double* g_color,
                             double* g_base, double* g_sh_rest, double* g_features,
                             double* g_weights, double* g_dirs) {
  std::vector<double> gw_rows;  // per-Gaussian weight-gradient rows, reduced in index order
  if (app == 1) {
    for (int k = 0; k < kNumW; ++k) g_weights[k] = 0;
  }
  const int na = num_active(deg);
  // process in chunks so the per-Gaussian dW rows stay small in memory but the final sum
  // runs in Gaussian-index order
  const int64_t chunk = 4096;
  if (app == 1) gw_rows.resize((size_t)chunk * kNumW);
  for (int64_t base = 0; base < n; base += chunk) {
    const int64_t m = std::min(chunk, n - base);
#pragma omp parallel for schedule(static)
    for (int64_t ii = 0; ii < m; ++ii) {
      const int64_t i = base + ii;
      for (int c = 0; c < 3; ++c) { g_base[3 * i + c] = 0; g_dirs[3 * i + c] = 0; }
      if (app == 0) for (int k = 0; k < 45; ++k) g_sh_rest[45 * i + k] = 0;
      if (app == 2) for (int k = 0; k < kSites * kSiteP; ++k) g_sh_rest[(size_t)kSites * kSiteP * i + k] = 0;
      if (app == 1) {
        for (int k = 0; k < kFeat; ++k) g_features[kFeat * i + k] = 0;
        std::fill(gw_rows.begin() + ii * kNumW, gw_rows.begin() + (ii + 1) * kNumW, 0.0);
      }
      if (mask && !mask[i]) continue;
      const double* d = dirs + 3 * i;
      double G[16][3];
      sh_basis_grad(d, G);
      if (app == 0) {
        double Y[16];
        sh_basis(d, Y);
        double A[3] = {0, 0, 0};
        for (int k = 1; k < na; ++k)
          for (int c = 0; c < 3; ++c) A[c] += Y[k] * sh_rest[(i * 15 + (k - 1)) * 3 + c];
        for (int c = 0; c < 3; ++c) {
          const double gp = color_act_grad(act, base_color[3 * i + c] + A[c]) * g_color[3 * i + c];
          g_base[3 * i + c] = gp;
          for (int k = 1; k < na; ++k) {
            g_sh_rest[(i * 15 + (k - 1)) * 3 + c] = Y[k] * gp;
            const double w = sh_rest[(i * 15 + (k - 1)) * 3 + c] * gp;
            for (int a = 0; a < 3; ++a) g_dirs[3 * i + a] += G[k][a] * w;
          }
        }
      } else if (app == 2) {   // Spherical Voronoi: sites in sh_rest, their gradients in g_sh_rest, [n,7,7]
        double A[3] = {0, 0, 0}, gp[3];
        SvState st;
        if (deg > 0) sv_forward(sh_rest + (size_t)i * kSites * kSiteP, d, A, st);
        for (int c = 0; c < 3; ++c) {
          gp[c] = color_act_grad(act, base_color[3 * i + c] + A[c]) * g_color[3 * i + c];
          g_base[3 * i + c] = gp[c];
        }
        if (deg > 0) sv_backward(sh_rest + (size_t)i * kSites * kSiteP, d, gp, st, A, g_sh_rest + (size_t)i * kSites * kSiteP, g_dirs + 3 * i);
      } else {
        if (deg == 0) {
          for (int c = 0; c < 3; ++c) {
            g_base[3 * i + c] = color_act_grad(act, base_color[3 * i + c]) * g_color[3 * i + c];
          }
          continue;
        }
        MlpState s;
        mlp_forward(weights, d, features + kFeat * i, deg, s);
        double* gw = gw_rows.data() + ii * kNumW;
        double gy[kOut], gh2[kHid], gh1[kHid], gx[kIn];
        for (int c = 0; c < 3; ++c) {
          const double gp = color_act_grad(act, base_color[3 * i + c] + s.A[c]) * g_color[3 * i + c];
          g_base[3 * i + c] = gp;
          gy[c] = gp * (1.0 - s.A[c] * s.A[c]);
        }
        for (int o = 0; o < kOut; ++o)
          for (int k = 0; k < kHid; ++k) gw[kW3 + o * kHid + k] = gy[o] * s.h2[k];
        for (int k = 0; k < kHid; ++k) {
          double a = 0;
          for (int o = 0; o < kOut; ++o) a += weights[kW3 + o * kHid + k] * gy[o];
          gh2[k] = s.h2[k] > 0 ? a : 0.0;
        }
        for (int o = 0; o < kHid; ++o)
          for (int k = 0; k < kHid; ++k) gw[kW2 + o * kHid + k] = gh2[o] * s.h1[k];
        for (int k = 0; k < kHid; ++k) {
          double a = 0;
          for (int o = 0; o < kHid; ++o) a += weights[kW2 + o * kHid + k] * gh2[o];
          gh1[k] = s.h1[k] > 0 ? a : 0.0;
        }
        for (int o = 0; o < kHid; ++o)
          for (int k = 0; k < kIn; ++k) gw[kW1 + o * kIn + k] = gh1[o] * s.x[k];
        for (int k = 0; k < kIn; ++k) {
          double a = 0;
          for (int o = 0; o < kHid; ++o) a += weights[kW1 + o * kIn + k] * gh1[o];
          gx[k] = a;
        }
        for (int j = 0; j < kFeat; ++j)
          g_features[kFeat * i + j] = gx[16 + 2 * j] * s.x[17 + 2 * j] - gx[17 + 2 * j] * s.x[16 + 2 * j];
        for (int k = 1; k < na; ++k)
          for (int a = 0; a < 3; ++a) g_dirs[3 * i + a] += gx[k] * G[k][a];
      }
    }
    if (app == 1)
      for (int64_t ii = 0; ii < m; ++ii)
        for (int k = 0; k < kNumW; ++k) g_weights[k] += gw_rows[ii * kNumW + k];
  }
}

// ---------------------------------------------------------------------------------------
// Integer stage on per-Gaussian values (centre, Cholesky factor of the conic, box half-extents and
// tau = 2 ln(255 o)) as produced by either side, in the precision F they come in (float for the
// GPU's values, double for the oracle's own).
//
// A Gaussian's instances are the tiles that its alpha >= 1/255 ellipse
//     (la dx + lb dy)^2 + (lc dy)^2 <= tau
// meets, found row of tiles by row of tiles inside the bounding tile rectangle: over the band of
// pixel-centre rows of one tile row the set is convex, so the tiles it meets are those between
// its leftmost and rightmost point in the band; the rightmost point is at the band end nearest
// to dy_r = -lb sqrt(tau/C)/lc (C = lb^2 + lc^2, where the ellipse's tangent is vertical), the
// leftmost at the end nearest to -dy_r.  tau and the band are padded (2e-5, 1e-5) so that
// rounding can only add a tile.  Each operation is rounded once, in this order.
// ---------------------------------------------------------------------------------------
}  // extern "C"

namespace {

template <class F>
struct Spans {
  F u, v, ila, lb, lc, taup, dys, eyp;
  int W, H;
  void setup(F u_, F v_, F la, F lb_, F lc_, F tau, int W_, int H_) {
    u = u_; v = v_; lb = lb_; lc = lc_; W = W_; H = H_;
    taup = tau * (F)1.00002f;
    const F rl = (F)1 / lc;
    ila = (F)1 / la;
    const F b2 = lb * lb, c2 = lc * lc;
    const F C = b2 + c2;
    const F q = taup / C;
    const F br = lb * rl;
    dys = br * std::sqrt(q);
    const F st = std::sqrt(taup) * rl;
    eyp = st * (F)1.00001f;
  }
  bool row(int ty, int tx0, int tx1, int& xa, int& xb) const {
    const F ylo = (F)(16 * ty) + (F)0.5, yhi = std::min((F)(16 * ty) + (F)15.5, (F)H - (F)0.5);
    const F da = std::max(ylo - v, -eyp), db = std::min(yhi - v, eyp);
    if (!(da <= db)) return false;
    const F dyR = std::min(std::max(-dys, da), db), dyL = std::min(std::max(dys, da), db);
    const F tR = lc * dyR, tL = lc * dyL;
    const F tR2 = tR * tR, tL2 = tL * tL;
    const F sR = std::sqrt(std::max(taup - tR2, (F)0)), sL = std::sqrt(std::max(taup - tL2, (F)0));
    const F bR = lb * dyR, bL = lb * dyL;
    const F xr = (sR - bR) * ila, xl = (-sL - bL) * ila;
    const F hi0 = u + xr, lo0 = u + xl;
    const F ihi = std::floor(hi0 - (F)0.5), ilo = std::ceil(lo0 - (F)0.5);
    if (!(ilo <= ihi) || ihi < 0 || ilo > (F)(W - 1)) return false;
    const int pa = (int)std::max(ilo, (F)0), pb = (int)std::min(ihi, (F)(W - 1));
    xa = std::max(pa >> 4, tx0);
    xb = std::min((pb >> 4) + 1, tx1);
    return xa < xb;
  }
};

template <class F>
int64_t tile_spans(int64_t n, const uint8_t* valid, const F* mean2d, const F* chol, const F* ext, int W, int H,
                   int32_t* rect, uint32_t* tiles_touched) {
  int64_t P = 0;
  for (int64_t i = 0; i < n; ++i) {
    for (int j = 0; j < 4; ++j) rect[4 * i + j] = 0;
    tiles_touched[i] = 0;
    if (!valid[i]) continue;
    int px[4]; bool empty;
    pixel_rect<F>(mean2d[2 * i], mean2d[2 * i + 1], ext[4 * i], ext[4 * i + 1], W, H, px, empty);
    if (empty) continue;
    int t[4];
    tile_rect(px, t);
    Spans<F> sp;
    sp.setup(mean2d[2 * i], mean2d[2 * i + 1], chol[3 * i], chol[3 * i + 1], chol[3 * i + 2], ext[4 * i + 2], W, H);
    uint32_t c = 0;
    for (int ty = t[1]; ty < t[3]; ++ty) {
      int xa, xb;
      if (sp.row(ty, t[0], t[2], xa, xb)) c += (uint32_t)(xb - xa);
    }
    if (c == 0) continue;
    for (int j = 0; j < 4; ++j) rect[4 * i + j] = t[j];
    tiles_touched[i] = c;
    P += c;
  }
  return P;
}

// Emit instances for Gaussian index ascending, tile rows top to bottom, tiles left to right;
// key = (tile_id << 32) | depth_bits; stable sort by key.
template <class F>
void sorted_instances(int64_t n, const int32_t* rect, const uint32_t* tiles_touched, const F* mean2d, const F* chol,
                      const F* ext, const uint32_t* depth_bits, int W, int H, int64_t P, uint64_t* keys,
                      uint32_t* vals) {
  const int gx = (W + kTile - 1) / kTile;
  std::vector<std::pair<uint64_t, uint32_t>> inst;
  inst.reserve((size_t)P);
  for (int64_t i = 0; i < n; ++i) {
    if (!tiles_touched[i]) continue;
    Spans<F> sp;
    sp.setup(mean2d[2 * i], mean2d[2 * i + 1], chol[3 * i], chol[3 * i + 1], chol[3 * i + 2], ext[4 * i + 2], W, H);
    for (int ty = rect[4 * i + 1]; ty < rect[4 * i + 3]; ++ty) {
      int xa, xb;
      if (!sp.row(ty, rect[4 * i], rect[4 * i + 2], xa, xb)) continue;
      for (int tx = xa; tx < xb; ++tx)
        inst.emplace_back(((uint64_t)(ty * gx + tx) << 32) | depth_bits[i], (uint32_t)i);
    }
  }
  std::stable_sort(inst.begin(), inst.end(),
                   [](const std::pair<uint64_t, uint32_t>& a, const std::pair<uint64_t, uint32_t>& b) {
                     return a.first < b.first;
                   });
  for (int64_t p = 0; p < P && p < (int64_t)inst.size(); ++p) { keys[p] = inst[p].first; vals[p] = inst[p].second; }
}

}  // namespace

extern "C" {

// mean2d [n,2], chol [n,3] = (la, lb, lc), ext [n,4] = (ex, ey, tau, -).  rect = (tx0, ty0, tx1, ty1),
// half open (all zero when no tile is met).  Return the pair count P.
int64_t gso_tile_spans_f32(int64_t n, const uint8_t* valid, const float* mean2d, const float* chol, const float* ext,
                           int W, int H, int32_t* rect, uint32_t* tiles_touched) {
  return tile_spans<float>(n, valid, mean2d, chol, ext, W, H, rect, tiles_touched);
}
int64_t gso_tile_spans_f64(int64_t n, const uint8_t* valid, const double* mean2d, const double* chol,
                           const double* ext, int W, int H, int32_t* rect, uint32_t* tiles_touched) {
  return tile_spans<double>(n, valid, mean2d, chol, ext, W, H, rect, tiles_touched);
}
void gso_sorted_instances_f32(int64_t n, const int32_t* rect, const uint32_t* tiles_touched, const float* mean2d,
                              const float* chol, const float* ext, const uint32_t* depth_bits, int W, int H,
                              int64_t P, uint64_t* keys, uint32_t* vals) {
  sorted_instances<float>(n, rect, tiles_touched, mean2d, chol, ext, depth_bits, W, H, P, keys, vals);
}
void gso_sorted_instances_f64(int64_t n, const int32_t* rect, const uint32_t* tiles_touched, const double* mean2d,
                              const double* chol, const double* ext, const uint32_t* depth_bits, int W, int H,
                              int64_t P, uint64_t* keys, uint32_t* vals) {
  sorted_instances<double>(n, rect, tiles_touched, mean2d, chol, ext, depth_bits, W, H, P, keys, vals);
}

void gso_tile_ranges(int64_t P, const uint64_t* keys, int num_tiles, uint32_t* ranges) {
  for (int t = 0; t < num_tiles; ++t) ranges[2 * t] = ranges[2 * t + 1] = 0;
  for (int64_t p = 0; p < P; ++p) {
    const uint32_t tile = (uint32_t)(keys[p] >> 32);
    if (p == 0 || tile != (uint32_t)(keys[p - 1] >> 32)) ranges[2 * tile] = (uint32_t)p;
    if (p == P - 1 || tile != (uint32_t)(keys[p + 1] >> 32)) ranges[2 * tile + 1] = (uint32_t)(p + 1);
  }
}

// ---------------------------------------------------------------------------------------
// Blend.  One pixel, one ordered list.  Returns through the pointers; `rec` (optional)
// records every composited entry for the backward pass.
// ---------------------------------------------------------------------------------------
// `ghost`: a pair the oracle did NOT composite although it sits within 1e-4 of a threshold, so an
// fp32 evaluation might; it only feeds the flip allowance of the backward.
struct Composited { uint32_t g; int pos; double alpha, T, power; bool clamped; bool ghost; };

// Half-width of the window around T (1 - alpha) = 1e-4 inside which a stop counts as one that an fp32 evaluation
// may take the other way: 1e-8 (a product of a few hundred fp32 factors, each carrying alpha's few ulp, is good to
// about 1e-4 relative, i.e. 1e-8 at the threshold).  A test may change it to measure what another width would flag.
static double g_stop_window = 1e-8;
void gso_set_stop_window(double w) { g_stop_window = w; }

static void blend_pixel(double px, double py, const uint32_t* list, int64_t len, const double* mean2d,
                        const double* conic, const double* opacity, const double* color,
                        const double bg[3], double out[3], double* final_T, uint32_t* n_contrib,
                        uint8_t* fragile, int32_t* fragile_pos, std::vector<Composited>* rec) {
  // fragile: some evaluated pair lies within 1e-4 (relative) of a blend threshold, so an fp32
  // evaluation may take the other branch; fragile_pos: list position of the first pair within
  // tolerance, or -1.  (fp32 alpha can be off by 1e-4 for footprints hundreds of pixels wide, and the
  // transmittance is a product of up to a thousand fp32 factors.)
  double T = 1.0, C[3] = {0, 0, 0};
  uint32_t last = 0;
  bool frag = false;
  int32_t fpos = -1;
  for (int64_t k = 0; k < len; ++k) {
    const uint32_t g = list[k];
    const double dx = px - mean2d[2 * g], dy = py - mean2d[2 * g + 1];
    const double power = -0.5 * (conic[3 * g] * dx * dx + conic[3 * g + 2] * dy * dy) - conic[3 * g + 1] * dx * dy;
    if (power > 0) continue;
    const double raw = opacity[g] * std::exp(power);
    const double alpha = std::min(kAlphaMax, raw);
    if (std::fabs(255.0 * alpha - 1.0) < 1e-4) frag = true;
    const bool near_alpha = std::fabs(255.0 * alpha - 1.0) < 1e-4;
    if (near_alpha && fpos < 0) fpos = (int32_t)k;
    // the 0.99 clamp switches the gradient of the pair on and off: also a branch fp32 may flip
    if (std::fabs(raw - kAlphaMax) < 1e-4 * kAlphaMax) { frag = true; if (fpos < 0) fpos = (int32_t)k; }
    if (alpha < kAlphaMin) {
      if (near_alpha && rec) rec->push_back({g, (int)k, alpha, T, power, false, true});
      continue;
    }
    const double Tn = T * (1.0 - alpha);
    if (std::fabs(Tn - kTmin) < g_stop_window) frag = true;
    const bool near_stop = std::fabs(Tn - kTmin) < g_stop_window;
    if (near_stop && fpos < 0) fpos = (int32_t)k;
    if (Tn < kTmin) {
      if (near_stop && rec) {
        // The stop is within tolerance: an fp32 evaluation may composite this pair and walk on.
        // Record what it would then add, as ghosts, until the transmittance is clearly below the
        // threshold.
        double Tg = T;
        for (int64_t kk = k; kk < len; ++kk) {
          const uint32_t gg = list[kk];
          const double ex = px - mean2d[2 * gg], ey = py - mean2d[2 * gg + 1];
          const double pw = -0.5 * (conic[3 * gg] * ex * ex + conic[3 * gg + 2] * ey * ey) - conic[3 * gg + 1] * ex * ey;
          if (pw > 0) continue;
          const double rw = opacity[gg] * std::exp(pw), al = std::min(kAlphaMax, rw);
          if (al < kAlphaMin) continue;
          const double Tgn = Tg * (1.0 - al);
          if (kk > k && Tgn < kTmin - g_stop_window) break;
          rec->push_back({gg, (int)kk, al, Tg, pw, rw > kAlphaMax, true});
          Tg = Tgn;
        }
      }
      break;
    }
    for (int c = 0; c < 3; ++c) C[c] += color[3 * g + c] * alpha * T;
    if (rec) rec->push_back({g, (int)k, alpha, T, power, raw > kAlphaMax, false});
    T = Tn;
    last = (uint32_t)(k + 1);
  }
  for (int c = 0; c < 3; ++c) out[c] = C[c] + T * bg[c];
  *final_T = T;
  *n_contrib = last;
  if (fragile) *fragile = frag ? 1 : 0;
  if (fragile_pos) *fragile_pos = fpos;
}

// One pixel's records, for the tests that pin the allowance logic: every entry the pixel composited and
// every ghost, in list order.  Returns the number of records (at most `cap` are written).
int64_t gso_blend_pixel_records(double px, double py, const uint32_t* list, int64_t len, const double* mean2d,
                                const double* conic, const double* opacity, const double* color, int64_t cap,
                                uint32_t* g, int32_t* pos, double* alpha, double* T, uint8_t* clamped,
                                uint8_t* ghost) {
  std::vector<Composited> rec;
  const double bg[3] = {0, 0, 0};
  double out[3], fT; uint32_t nc; uint8_t frag; int32_t fpos;
  blend_pixel(px, py, list, len, mean2d, conic, opacity, color, bg, out, &fT, &nc, &frag, &fpos, &rec);
  for (int64_t k = 0; k < (int64_t)rec.size() && k < cap; ++k) {
    g[k] = rec[k].g; pos[k] = rec[k].pos; alpha[k] = rec[k].alpha; T[k] = rec[k].T;
    clamped[k] = rec[k].clamped ? 1 : 0; ghost[k] = rec[k].ghost ? 1 : 0;
  }
  return (int64_t)rec.size();
}

// Tiled forward: image[3,H,W], final_T[H,W], n_contrib[H,W], fragile[H,W] (u8), fragile_pos[H,W].
void gso_blend_forward(int W, int H, const double* bg, const uint32_t* vals, const uint32_t* ranges,
                       const double* mean2d, const double* conic, const double* opacity,
                       const double* color, double* image, double* final_T, uint32_t* n_contrib,
                       uint8_t* fragile, int32_t* fragile_pos) {
  const int gx = (W + kTile - 1) / kTile, gy = (H + kTile - 1) / kTile;
#pragma omp parallel for schedule(dynamic, 1)
  for (int tile = 0; tile < gx * gy; ++tile) {
    const int tx = tile % gx, ty = tile / gx;
    const uint32_t s = ranges[2 * tile], e = ranges[2 * tile + 1];
    for (int j = ty * kTile; j < std::min(H, (ty + 1) * kTile); ++j)
      for (int i = tx * kTile; i < std::min(W, (tx + 1) * kTile); ++i) {
        double out[3];
        blend_pixel(i + 0.5, j + 0.5, vals + s, (int64_t)e - s, mean2d, conic, opacity, color, bg, out,
                    &final_T[(size_t)j * W + i], &n_contrib[(size_t)j * W + i],
                    fragile ? &fragile[(size_t)j * W + i] : nullptr,
                    fragile_pos ? &fragile_pos[(size_t)j * W + i] : nullptr, nullptr);
        for (int c = 0; c < 3; ++c) image[((size_t)c * H + j) * W + i] = out[c];
      }
  }
}

// The plain definition: every visible Gaussian, ordered by (depth_bits, index), every pixel.
void gso_blend_brute(int64_t n, int W, int H, const double* bg, const uint8_t* visible,
                     const uint32_t* depth_bits, const double* mean2d, const double* conic,
                     const double* opacity, const double* color, double* image, double* final_T) {
  std::vector<uint32_t> order;
  for (int64_t i = 0; i < n; ++i) if (visible[i]) order.push_back((uint32_t)i);
  std::stable_sort(order.begin(), order.end(),
                   [&](uint32_t a, uint32_t b) { return depth_bits[a] < depth_bits[b]; });
#pragma omp parallel for schedule(static)
  for (int j = 0; j < H; ++j)
    for (int i = 0; i < W; ++i) {
      double out[3]; uint32_t nc;
      blend_pixel(i + 0.5, j + 0.5, order.data(), (int64_t)order.size(), mean2d, conic, opacity, color,
                  bg, out, &final_T[(size_t)j * W + i], &nc, nullptr, nullptr, nullptr);
      for (int c = 0; c < 3; ++c) image[((size_t)c * H + j) * W + i] = out[c];
    }
}

// Backward of the blend for L with upstream G = dL/dimage [3,H,W].
// Outputs per Gaussian: g_color[n,3], g_opacity[n], g_conic[n,3] (A,B,C), g_mean2d[n,2];
// abs_sum (optional, [n,9] = colour3, opacity, conic3, mean2): the sums of the absolute values of
// the accumulated terms (conditioning of the fp32 summation).  flip_sum (optional, [n,9]): the
// absolute values of the terms that an fp32 evaluation could add, drop or rescale because some pair
// of the pixel sits within 1e-4 of a blend threshold - that pair and every entry behind it.
void gso_blend_backward(int64_t n, int W, int H, const double* bg, int64_t P, const uint32_t* vals,
                        const uint32_t* ranges, const double* mean2d, const double* conic,
                        const double* opacity, const double* color, const double* G,
                        double* g_color, double* g_opacity, double* g_conic, double* g_mean2d,
                        double* abs_sum, double* flip_sum) {
  const int gx = (W + kTile - 1) / kTile, gy = (H + kTile - 1) / kTile;
  std::vector<double> inst((size_t)P * 9, 0.0), inst_abs(abs_sum ? (size_t)P * 9 : 0, 0.0),
      inst_flip(flip_sum ? (size_t)P * 9 : 0, 0.0);
#pragma omp parallel for schedule(dynamic, 1)
  for (int tile = 0; tile < gx * gy; ++tile) {
    const int tx = tile % gx, ty = tile / gx;
    const uint32_t s = ranges[2 * tile], e = ranges[2 * tile + 1];
    std::vector<Composited> rec;
    for (int j = ty * kTile; j < std::min(H, (ty + 1) * kTile); ++j)
      for (int i = tx * kTile; i < std::min(W, (tx + 1) * kTile); ++i) {
        rec.clear();
        double out[3], fT; uint32_t nc; int32_t fpos = -1;
        const double px = i + 0.5, py = j + 0.5;
        blend_pixel(px, py, vals + s, (int64_t)e - s, mean2d, conic, opacity, color, bg, out, &fT, &nc,
                    nullptr, &fpos, &rec);
        double Gp[3];
        for (int c = 0; c < 3; ++c) Gp[c] = G[((size_t)c * H + j) * W + i];
        // S = light arriving from behind the current entry, built back to front
        double S[3] = {fT * bg[0], fT * bg[1], fT * bg[2]};
        for (int k = (int)rec.size() - 1; k >= 0; --k) {
          const Composited& r = rec[k];
          const uint32_t g = r.g;
          double* acc = inst.data() + ((size_t)s + r.pos) * 9;
          double* aab = abs_sum ? inst_abs.data() + ((size_t)s + r.pos) * 9 : nullptr;
          double* afl = (flip_sum && fpos >= 0 && r.pos >= fpos) ? inst_flip.data() + ((size_t)s + r.pos) * 9 : nullptr;
          bool real = !r.ghost;
          auto add = [&](int slot, double v) {
            if (real) { acc[slot] += v; if (aab) aab[slot] += std::fabs(v); }
            if (afl) afl[slot] += std::fabs(v);
          };
          double dalpha = 0;
          for (int c = 0; c < 3; ++c) {
            add(c, r.alpha * r.T * Gp[c]);
            dalpha += Gp[c] * (r.T * color[3 * g + c] - S[c] / (1.0 - r.alpha));
          }
          const bool near_clamp = std::fabs(opacity[g] * std::exp(r.power) - kAlphaMax) < 1e-4 * kAlphaMax;
          if (!r.clamped || near_clamp) {
            if (r.clamped) real = false;   // clamped here, but fp32 may not clamp: flip allowance only
            const double dpower = r.alpha * dalpha;
            const double dx = px - mean2d[2 * g], dy = py - mean2d[2 * g + 1];
            add(3, std::exp(r.power) * dalpha);
            add(4, -0.5 * dx * dx * dpower);
            add(5, -dx * dy * dpower);
            add(6, -0.5 * dy * dy * dpower);
            // d power / d mean = +(A dx + B dy, B dx + C dy)
            add(7, dpower * (conic[3 * g] * dx + conic[3 * g + 1] * dy));
            add(8, dpower * (conic[3 * g + 1] * dx + conic[3 * g + 2] * dy));
          }
          if (!r.ghost) for (int c = 0; c < 3; ++c) S[c] += color[3 * g + c] * r.alpha * r.T;
        }
      }
  }
  for (int64_t i = 0; i < n; ++i) {
    for (int c = 0; c < 3; ++c) { g_color[3 * i + c] = 0; g_conic[3 * i + c] = 0; }
    g_opacity[i] = 0; g_mean2d[2 * i] = g_mean2d[2 * i + 1] = 0;
    if (abs_sum) for (int c = 0; c < 9; ++c) abs_sum[9 * i + c] = 0;
    if (flip_sum) for (int c = 0; c < 9; ++c) flip_sum[9 * i + c] = 0;
  }
  for (int64_t p = 0; p < P; ++p) {
    const uint32_t g = vals[p];
    const double* a = inst.data() + (size_t)p * 9;
    for (int c = 0; c < 3; ++c) g_color[3 * g + c] += a[c];
    g_opacity[g] += a[3];
    for (int c = 0; c < 3; ++c) g_conic[3 * g + c] += a[4 + c];
    g_mean2d[2 * g] += a[7]; g_mean2d[2 * g + 1] += a[8];
    if (abs_sum) for (int c = 0; c < 9; ++c) abs_sum[9 * g + c] += inst_abs[(size_t)p * 9 + c];
    if (flip_sum) for (int c = 0; c < 9; ++c) flip_sum[9 * g + c] += inst_flip[(size_t)p * 9 + c];
  }
}

// ---------------------------------------------------------------------------------------
// Backward of the projection: 2D gradients (g_mean2d, g_conic, g_opacity) and the direction
// gradient g_dir (from the appearance backward) -> gradients of means, log_scales, quats,
// opacity_logits.  Rows with visible == 0 get exact zeros.
// ---------------------------------------------------------------------------------------
void gso_preprocess_backward(int64_t n, const double* means, const double* log_scales,
                             const double* quats, const double* opacity_logits, const double* cam_,
                             const uint8_t* visible, const double* g_mean2d, const double* g_conic,
                             const double* g_opacity, const double* g_dir, double* g_means,
                             double* g_log_scales, double* g_quats, double* g_logits) {
  const Cam cam = read_cam(cam_);
  double oc[3];
  for (int j = 0; j < 3; ++j)
    oc[j] = -(cam.R[0 + j] * cam.t[0] + cam.R[3 + j] * cam.t[1] + cam.R[6 + j] * cam.t[2]);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    for (int j = 0; j < 3; ++j) { g_means[3 * i + j] = 0; g_log_scales[3 * i + j] = 0; }
    for (int j = 0; j < 4; ++j) g_quats[4 * i + j] = 0;
    g_logits[i] = 0;
    if (!visible[i]) continue;
    const double* mu = means + 3 * i;
    // ---- recompute the forward quantities
    const double* q = quats + 4 * i;
    const double qn = std::sqrt(q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3]);
    const double qh[4] = {q[0] / qn, q[1] / qn, q[2] / qn, q[3] / qn};
    double R[9], s[3], M[9], S[9];
    quat_to_rot(qh, R);
    for (int k = 0; k < 3; ++k) s[k] = std::exp(log_scales[3 * i + k]);
    for (int r = 0; r < 3; ++r) for (int k = 0; k < 3; ++k) M[3 * r + k] = R[3 * r + k] * s[k];
    for (int r = 0; r < 3; ++r)
      for (int c = 0; c < 3; ++c) {
        double a = 0;
        for (int k = 0; k < 3; ++k) a += M[3 * r + k] * M[3 * c + k];
        S[3 * r + c] = a;
      }
    double t[3];
    for (int r = 0; r < 3; ++r)
      t[r] = cam.R[3 * r] * mu[0] + cam.R[3 * r + 1] * mu[1] + cam.R[3 * r + 2] * mu[2] + cam.t[r];
    const double limx = 1.3 * (cam.W / 2.0) / cam.fx, limy = 1.3 * (cam.H / 2.0) / cam.fy;
    const double rx = t[0] / t[2], ry = t[1] / t[2];
    const bool clx = rx < -limx || rx > limx, cly = ry < -limy || ry > limy;
    const double txc = t[2] * std::min(limx, std::max(-limx, rx));
    const double tyc = t[2] * std::min(limy, std::max(-limy, ry));
    const double z2 = t[2] * t[2];
    const double J[6] = {cam.fx / t[2], 0, -cam.fx * txc / z2, 0, cam.fy / t[2], -cam.fy * tyc / z2};
    double T[6];
    for (int r = 0; r < 2; ++r)
      for (int c = 0; c < 3; ++c)
        T[3 * r + c] = J[3 * r] * cam.R[c] + J[3 * r + 1] * cam.R[3 + c] + J[3 * r + 2] * cam.R[6 + c];
    double TS[6];
    for (int r = 0; r < 2; ++r)
      for (int c = 0; c < 3; ++c)
        TS[3 * r + c] = T[3 * r] * S[c] + T[3 * r + 1] * S[3 + c] + T[3 * r + 2] * S[6 + c];
    const double a = TS[0] * T[0] + TS[1] * T[1] + TS[2] * T[2] + kDilation;
    const double b = TS[0] * T[3] + TS[1] * T[4] + TS[2] * T[5];
    const double c = TS[3] * T[3] + TS[4] * T[4] + TS[5] * T[5] + kDilation;
    const double det = a * c - b * b;
    const double Q[4] = {c / det, -b / det, -b / det, a / det};
    // ---- conic -> 2D covariance:  G_cov = -Q G_Q Q, G_Q = [[gA, gB/2], [gB/2, gC]]
    const double GQ[4] = {g_conic[3 * i], 0.5 * g_conic[3 * i + 1], 0.5 * g_conic[3 * i + 1], g_conic[3 * i + 2]};
    double QG[4], Gc[4];
    for (int r = 0; r < 2; ++r) for (int k = 0; k < 2; ++k) QG[2 * r + k] = Q[2 * r] * GQ[k] + Q[2 * r + 1] * GQ[2 + k];
    for (int r = 0; r < 2; ++r) for (int k = 0; k < 2; ++k) Gc[2 * r + k] = -(QG[2 * r] * Q[k] + QG[2 * r + 1] * Q[2 + k]);
    // ---- cov = T Sigma T^T + 0.3 I:  G_Sigma = T^T G_cov T,  G_T = 2 G_cov T Sigma
    double GcT[6];
    for (int r = 0; r < 2; ++r) for (int k = 0; k < 3; ++k) GcT[3 * r + k] = Gc[2 * r] * T[k] + Gc[2 * r + 1] * T[3 + k];
    double GS[9];
    for (int r = 0; r < 3; ++r) for (int k = 0; k < 3; ++k) GS[3 * r + k] = T[r] * GcT[k] + T[3 + r] * GcT[3 + k];
    double GT[6];
    for (int r = 0; r < 2; ++r)
      for (int k = 0; k < 3; ++k)
        GT[3 * r + k] = 2.0 * (GcT[3 * r] * S[k] + GcT[3 * r + 1] * S[3 + k] + GcT[3 * r + 2] * S[6 + k]);
    // ---- T = J R_c:  G_J = G_T R_c^T
    double GJ[6];
    for (int r = 0; r < 2; ++r)
      for (int k = 0; k < 3; ++k)
        GJ[3 * r + k] = GT[3 * r] * cam.R[3 * k] + GT[3 * r + 1] * cam.R[3 * k + 1] + GT[3 * r + 2] * cam.R[3 * k + 2];
    // ---- J and mean2d -> t
    double gt[3] = {0, 0, 0};
    const double gu = g_mean2d[2 * i], gv = g_mean2d[2 * i + 1];
    gt[0] += gu * cam.fx / t[2];
    gt[1] += gv * cam.fy / t[2];
    gt[2] += -(gu * cam.fx * t[0] + gv * cam.fy * t[1]) / z2;
    gt[2] += GJ[0] * (-cam.fx / z2) + GJ[4] * (-cam.fy / z2);
    if (!clx) { gt[0] += GJ[2] * (-cam.fx / z2); gt[2] += GJ[2] * (2.0 * cam.fx * t[0] / (z2 * t[2])); }
    else      { gt[2] += GJ[2] * (-J[2] / t[2]); }
    if (!cly) { gt[1] += GJ[5] * (-cam.fy / z2); gt[2] += GJ[5] * (2.0 * cam.fy * t[1] / (z2 * t[2])); }
    else      { gt[2] += GJ[5] * (-J[5] / t[2]); }
    double gmu[3];
    for (int k = 0; k < 3; ++k) gmu[k] = cam.R[k] * gt[0] + cam.R[3 + k] * gt[1] + cam.R[6 + k] * gt[2];
    // ---- direction d = (mu - o_c)/|mu - o_c|
    double dv[3] = {mu[0] - oc[0], mu[1] - oc[1], mu[2] - oc[2]};
    const double dn = std::sqrt(dv[0] * dv[0] + dv[1] * dv[1] + dv[2] * dv[2]);
    const double d[3] = {dv[0] / dn, dv[1] / dn, dv[2] / dn};
    const double* gd = g_dir + 3 * i;
    const double dot = d[0] * gd[0] + d[1] * gd[1] + d[2] * gd[2];
    for (int k = 0; k < 3; ++k) gmu[k] += (gd[k] - d[k] * dot) / dn;
    for (int k = 0; k < 3; ++k) g_means[3 * i + k] = gmu[k];
    // ---- Sigma = M M^T:  G_M = 2 G_Sigma M
    double GM[9];
    for (int r = 0; r < 3; ++r)
      for (int k = 0; k < 3; ++k)
        GM[3 * r + k] = 2.0 * (GS[3 * r] * M[k] + GS[3 * r + 1] * M[3 + k] + GS[3 * r + 2] * M[6 + k]);
    double D[9];  // dL/dR
    for (int k = 0; k < 3; ++k) {
      double gs = 0;
      for (int r = 0; r < 3; ++r) { gs += GM[3 * r + k] * R[3 * r + k]; D[3 * r + k] = GM[3 * r + k] * s[k]; }
      g_log_scales[3 * i + k] = s[k] * gs;
    }
    const double r_ = qh[0], x = qh[1], y = qh[2], z = qh[3];
    double gq[4];
    gq[0] = 2 * (-z * D[1] + y * D[2] + z * D[3] - x * D[5] - y * D[6] + x * D[7]);
    gq[1] = 2 * (y * D[1] + z * D[2] + y * D[3] - 2 * x * D[4] - r_ * D[5] + z * D[6] + r_ * D[7] - 2 * x * D[8]);
    gq[2] = 2 * (-2 * y * D[0] + x * D[1] + r_ * D[2] + x * D[3] + z * D[5] - r_ * D[6] + z * D[7] - 2 * y * D[8]);
    gq[3] = 2 * (-2 * z * D[0] - r_ * D[1] + x * D[2] + r_ * D[3] - 2 * z * D[4] + y * D[5] + x * D[6] + y * D[7]);
    const double qdot = qh[0] * gq[0] + qh[1] * gq[1] + qh[2] * gq[2] + qh[3] * gq[3];
    for (int k = 0; k < 4; ++k) g_quats[4 * i + k] = (gq[k] - qh[k] * qdot) / qn;
    const double o = 1.0 / (1.0 + std::exp(-opacity_logits[i]));
    g_logits[i] = g_opacity[i] * o * (1.0 - o);
  }
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// The decoder with its architecture as a parameter (App. D, architecture table): `layers` hidden layers
// (1..3) of `hidden` neurons (16 or 32), ReLU, no biases, three tanh outputs; input = 16 SH basis values of
// the direction (masked by the active degree) followed by 16 feature inputs: nfeat = 8 features as
// (sin f_j, cos f_j) pairs (Eq. 6, k = 1), or nfeat = 16 raw features without frequency encoding.
// Weights: W_1[hidden][32], then layers - 1 matrices [hidden][hidden], then W_out[3][hidden], row-major.
// A second, independent statement of Eq. 5-7: for hidden = 16, layers = 2, nfeat = 8 it must agree with
// the fixed-size decoder above.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kMaxHid = 32, kMaxLayers = 3;
struct DecState { double x[32], h[kMaxLayers][kMaxHid], A[3]; };
int dec_num_weights(int hidden, int layers) { return 32 * hidden + (layers - 1) * hidden * hidden + 3 * hidden; }
void dec_inputs(const double* d, const double* f, int nfeat, int deg, double x[32]) {
  double Y[16];
  sh_basis(d, Y);
  const int na = num_active(deg);
  for (int k = 0; k < 16; ++k) x[k] = k < na ? Y[k] : 0.0;
  if (nfeat == 8)
    for (int j = 0; j < 8; ++j) { x[16 + 2 * j] = std::sin(f[j]); x[17 + 2 * j] = std::cos(f[j]); }
  else
    for (int j = 0; j < 16; ++j) x[16 + j] = f[j];
}
void dec_forward(const double* W, int hidden, int layers, const double x[32], DecState& s) {
  const double* w = W;
  const double* in = x;
  int nin = 32;
  for (int l = 0; l < layers; ++l) {
    for (int o = 0; o < hidden; ++o) {
      double a = 0;
      for (int i = 0; i < nin; ++i) a += w[o * nin + i] * in[i];
      s.h[l][o] = a > 0 ? a : 0;
    }
    w += hidden * nin; in = s.h[l]; nin = hidden;
  }
  for (int o = 0; o < 3; ++o) {
    double a = 0;
    for (int i = 0; i < hidden; ++i) a += w[o * hidden + i] * in[i];
    s.A[o] = std::tanh(a);
  }
}
}  // namespace

extern "C" {
int gso_decoder_num_weights(int hidden, int layers) { return dec_num_weights(hidden, layers); }
// Multiply-accumulates per Gaussian; fold = 1: the 17 view-independent columns of the first layer are
// pre-multiplied per Gaussian (only worthwhile while hidden <= 16, App. C.3).
int gso_decoder_macs(int hidden, int layers, int fold) {
  return (fold ? 16 : 32) * hidden + (layers - 1) * hidden * hidden + 3 * hidden;
}
void gso_decoder_forward(int64_t n, int hidden, int layers, int nfeat, int deg, int act, const double* base_color,
                         const double* features, const double* weights, const double* dirs, double* color) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    DecState s;
    s.A[0] = s.A[1] = s.A[2] = 0;
    if (deg > 0) {
      double x[32];
      dec_inputs(dirs + 3 * i, features + (size_t)nfeat * i, nfeat, deg, x);
      dec_forward(weights, hidden, layers, x, s);
    }
    for (int c = 0; c < 3; ++c) color[3 * i + c] = color_act(act, base_color[3 * i + c] + s.A[c]);
  }
}
// g_weights is the sum over the Gaussians in index order.
void gso_decoder_backward(int64_t n, int hidden, int layers, int nfeat, int deg, int act, const double* base_color,
                          const double* features, const double* weights, const double* dirs, const double* g_color,
                          double* g_base, double* g_features, double* g_weights, double* g_dirs) {
  const int nw = dec_num_weights(hidden, layers);
  for (int k = 0; k < nw; ++k) g_weights[k] = 0;
  const int na = num_active(deg);
  for (int64_t i = 0; i < n; ++i) {
    for (int c = 0; c < 3; ++c) g_dirs[3 * i + c] = 0;
    for (int j = 0; j < nfeat; ++j) g_features[(size_t)nfeat * i + j] = 0;
    if (deg == 0) {
      for (int c = 0; c < 3; ++c) g_base[3 * i + c] = color_act_grad(act, base_color[3 * i + c]) * g_color[3 * i + c];
      continue;
    }
    DecState s;
    double x[32];
    dec_inputs(dirs + 3 * i, features + (size_t)nfeat * i, nfeat, deg, x);
    dec_forward(weights, hidden, layers, x, s);
    double g_out[kMaxHid], g_in[kMaxHid > 32 ? kMaxHid : 32];
    for (int c = 0; c < 3; ++c) {
      const double gp = color_act_grad(act, base_color[3 * i + c] + s.A[c]) * g_color[3 * i + c];
      g_base[3 * i + c] = gp;
      g_out[c] = gp * (1.0 - s.A[c] * s.A[c]);
    }
    // walk the layers from the output back: offsets of each matrix
    int off[kMaxLayers + 1];
    off[0] = 0;
    for (int l = 1; l <= layers; ++l) off[l] = off[l - 1] + hidden * (l == 1 ? 32 : hidden);
    int nout = 3;
    for (int l = layers; l >= 0; --l) {
      const double* in = l == 0 ? x : s.h[l - 1];
      const int nin = l == 0 ? 32 : hidden;
      const double* w = weights + off[l];
      double* gw = g_weights + off[l];
      for (int o = 0; o < nout; ++o)
        for (int k = 0; k < nin; ++k) gw[o * nin + k] += g_out[o] * in[k];
      for (int k = 0; k < nin; ++k) {
        double a = 0;
        for (int o = 0; o < nout; ++o) a += w[o * nin + k] * g_out[o];
        g_in[k] = (l == 0 || in[k] > 0) ? a : 0.0;     // ReLU of the layer below (the inputs have none)
      }
      for (int k = 0; k < nin; ++k) g_out[k] = g_in[k];
      nout = hidden;
      if (l == 0) break;
    }
    // g_out now holds dL/dx[0..31]
    if (nfeat == 8)
      for (int j = 0; j < 8; ++j) g_features[8 * i + j] = g_out[16 + 2 * j] * x[17 + 2 * j] - g_out[17 + 2 * j] * x[16 + 2 * j];
    else
      for (int j = 0; j < 16; ++j) g_features[16 * i + j] = g_out[16 + j];
    double G[16][3];
    sh_basis_grad(dirs + 3 * i, G);
    for (int k = 1; k < na; ++k)
      for (int a = 0; a < 3; ++a) g_dirs[3 * i + a] += G[k][a] * g_out[k];
  }
}
}

extern "C" {
double gso_color_act(int act, double x) { return color_act(act, x); }
double gso_color_act_grad(int act, double x) { return color_act_grad(act, x); }
}
