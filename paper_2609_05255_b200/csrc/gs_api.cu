// The C ABI: argument validation, workspace carving and kernel launches.  No arithmetic of the
// method lives here.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gs_device.cuh"

struct StageRecord { int stage; int launches; cudaEvent_t begin, end; };

struct GsContext {
  int device;
  int num_sms;
  unsigned long long *d_counter;      // device: [0] instance counter of the last gs_preprocess, [2] set when a device-counted
                                      // view overflowed its capacity, [3] set when a bounded device-side wait ran out,
                                      // [4..7] the four words of gs_profile_blend_counts
  unsigned long long *h_counter;      // pinned host mirror
  float *d_w_partials;                // device: per-CTA partial sums of the decoder gradient ([kWgradBlocks, 816];
                                      // sized for the decoder variants' largest case as well)
  char error[256];
  int decoder_engine;                 // GsDecoderEngine of the separate-pass forward
  bool profiling;
  std::vector<StageRecord> records;   // stage timings since the last collect
  std::vector<cudaEvent_t> free_events;
};

namespace {

using namespace gs;

GsStatus fail(GsContext *ctx, GsStatus code, const char *fmt, const char *detail = "") {
  if (ctx) snprintf(ctx->error, sizeof(ctx->error), fmt, detail);
  return code;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool bad_ptr(const void *p) { return p == nullptr || !aligned16(p); }

GsStatus check_cuda(GsContext *ctx, cudaError_t e, const char *what) {
  if (e == cudaSuccess) return GS_OK;
  if (ctx) snprintf(ctx->error, sizeof(ctx->error), "%s: %s", what, cudaGetErrorString(e));
  return GS_ERR_CUDA;
}

const char *const kStageNames[] = {"preprocess_fwd", "depth_sort", "tile_offsets", "keygen", "tile_sort", "tile_ranges",
                                   "blend_fwd", "blend_bwd", "preprocess_bwd", "appearance_fwd", "appearance_bwd",
                                   "adam", "prepass"};
static_assert(sizeof(kStageNames) / sizeof(kStageNames[0]) == GS_NUM_STAGES, "one name per stage");

// Brackets one stage with events, and with an NVTX range for a tracing tool, when profiling is on.
struct StageTimer {
  GsContext *ctx; cudaStream_t st; StageRecord rec; bool active;
  static cudaEvent_t get_event(GsContext *ctx) {
    if (!ctx->free_events.empty()) { cudaEvent_t e = ctx->free_events.back(); ctx->free_events.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
  }
  StageTimer(GsContext *c, int stage, cudaStream_t s) : ctx(c), st(s), active(c->profiling && c->records.size() < 4096) {
    if (!active) return;
    rec.stage = stage; rec.launches = 0;
    rec.begin = get_event(ctx); rec.end = get_event(ctx);
    if (stage >= 0 && stage < (int)(sizeof(kStageNames) / sizeof(kStageNames[0]))) nvtxRangePushA(kStageNames[stage]);
    else nvtxRangePushA("gs");
    cudaEventRecord(rec.begin, st);
  }
  void done(int launches) {
    if (!active) return;
    rec.launches = launches;
    cudaEventRecord(rec.end, st);
    nvtxRangePop();
    ctx->records.push_back(rec);
  }
};

bool camera_ok(const GsCamera *c) {
  if (!c || c->width <= 0 || c->height <= 0) return false;
  if (!(c->fx > 0.f) || !(c->fy > 0.f)) return false;
  const int64_t gx = (c->width + GS_TILE - 1) / GS_TILE, gy = (c->height + GS_TILE - 1) / GS_TILE;
  if (gx > 65535 || gy > 65535 || ((gx + 3) / 4) * ((gy + 3) / 4) > 65536) return false;   // rect is u16; a cell id takes 16 bits
  return true;
}

CamDev make_cam(const GsCamera *c) {
  CamDev d;
  d.W = c->width; d.H = c->height;
  d.gx = (c->width + GS_TILE - 1) / GS_TILE; d.gy = (c->height + GS_TILE - 1) / GS_TILE;
  d.cgx = (d.gx + 3) / 4; d.cgy = (d.gy + 3) / 4;
  d.fx = c->fx; d.fy = c->fy; d.cx = c->cx; d.cy = c->cy;
  for (int r = 0; r < 3; ++r) {
    for (int k = 0; k < 3; ++k) d.R[3 * r + k] = c->w2c[4 * r + k];
    d.t[r] = c->w2c[4 * r + 3];
  }
  for (int k = 0; k < 3; ++k)
    d.oc[k] = (float)-((double)d.R[k] * d.t[0] + (double)d.R[3 + k] * d.t[1] + (double)d.R[6 + k] * d.t[2]);
  d.near_plane = c->near_plane; d.far_plane = c->far_plane;
  d.limx = (float)(1.3 * (c->width / 2.0) / c->fx);
  d.limy = (float)(1.3 * (c->height / 2.0) / c->fy);
  for (int k = 0; k < 3; ++k) d.bg[k] = c->background[k];
  return d;
}

struct DecoderArch { int hidden, layers, nfeat; };
DecoderArch decoder_arch(const GsScene *s) {
  return {s->mlp_hidden ? s->mlp_hidden : 16, s->mlp_layers ? s->mlp_layers : 2, s->num_features ? s->num_features : 8};
}
bool default_decoder(const GsScene *s) {
  const DecoderArch d = decoder_arch(s);
  return s->app != GS_APP_NEURAL || (d.hidden == 16 && d.layers == 2 && d.nfeat == 8);
}
// The template instance a scene's appearance kernels run as.
int kernel_app(const GsScene *s) {
  return s->app == GS_APP_NEURAL && s->decoder_precision == GS_DECODER_HALF ? kAppNeuralHalf : s->app;
}
// The rendering step with the appearance as passes of its own (asked for, or the only way for a decoder variant).
bool unfused(const GsScene *s) { return s->separate_pass != 0 || !default_decoder(s); }

AppearanceArgs appearance_args(GsContext *ctx, const GsScene *scene) {
  AppearanceArgs a;
  memset(&a, 0, sizeof(a));
  a.timeout = ctx->d_counter + 3;
  a.engine = ctx->decoder_engine;
  a.n = scene->n; a.deg = scene->active_degree; a.act = scene->color_activation;
  a.base_color = scene->base_color; a.sh_rest = scene->app == GS_APP_SV ? scene->sv_sites : scene->sh_rest;
  a.features = reinterpret_cast<const __half *>(scene->features);
  a.weights = reinterpret_cast<const __half *>(scene->mlp_weights);
  return a;
}
int run_appearance_fwd(const GsScene *scene, const AppearanceArgs &a, cudaStream_t s) {
  const DecoderArch d = decoder_arch(scene);
  return default_decoder(scene) ? launch_appearance_fwd(kernel_app(scene), a, s) : launch_variant_fwd(d.hidden, d.layers, d.nfeat, a, s);
}
int run_appearance_bwd(const GsScene *scene, const AppearanceArgs &a, cudaStream_t s) {
  const DecoderArch d = decoder_arch(scene);
  return default_decoder(scene) ? launch_appearance_bwd(kernel_app(scene), a, s) : launch_variant_bwd(d.hidden, d.layers, d.nfeat, a, s);
}

GsStatus scene_appearance_ok(GsContext *ctx, const GsScene *s) {
  if (s->app != GS_APP_SH && s->app != GS_APP_NEURAL && s->app != GS_APP_SV) return fail(ctx, GS_ERR_INVALID_ARG, "unknown appearance model");
  if (s->active_degree < 0 || s->active_degree > 3) return fail(ctx, GS_ERR_INVALID_ARG, "active_degree must be 0..3");
  if (s->color_activation < GS_ACT_RELU || s->color_activation > GS_ACT_HARD_SIGMOID)
    return fail(ctx, GS_ERR_INVALID_ARG, "unknown colour activation");
  if (s->decoder_precision != GS_DECODER_SPLIT && s->decoder_precision != GS_DECODER_HALF)
    return fail(ctx, GS_ERR_INVALID_ARG, "unknown decoder precision");
  if (s->n < 0) return fail(ctx, GS_ERR_INVALID_ARG, "n < 0");
  if (s->n >= ((int64_t)1 << 31)) return fail(ctx, GS_ERR_CAPACITY, "n must stay below 2^31 (32-bit Gaussian ids and grids)");
  if (s->app == GS_APP_NEURAL) {
    const DecoderArch d = decoder_arch(s);
    if ((d.hidden != 16 && d.hidden != 32) || d.layers < 1 || d.layers > 3 || (d.nfeat != 8 && d.nfeat != 16))
      return fail(ctx, GS_ERR_INVALID_ARG, "decoder must have 1..3 hidden layers of 16 or 32 neurons and 8 or 16 features");
  }
  if (s->n == 0) return GS_OK;
  if (bad_ptr(s->base_color)) return fail(ctx, GS_ERR_INVALID_ARG, "base_color is NULL or misaligned");
  if (s->app == GS_APP_SH && bad_ptr(s->sh_rest)) return fail(ctx, GS_ERR_INVALID_ARG, "sh_rest is NULL or misaligned");
  if (s->app == GS_APP_SV && bad_ptr(s->sv_sites)) return fail(ctx, GS_ERR_INVALID_ARG, "sv_sites is NULL or misaligned");
  if (s->app == GS_APP_NEURAL && (bad_ptr(s->features) || bad_ptr(s->mlp_weights)))
    return fail(ctx, GS_ERR_INVALID_ARG, "features / mlp_weights is NULL or misaligned");
  return GS_OK;
}

GsStatus scene_ok(GsContext *ctx, const GsScene *s) {
  if (!s) return fail(ctx, GS_ERR_INVALID_ARG, "scene is NULL");
  GsStatus st = scene_appearance_ok(ctx, s);
  if (st != GS_OK) return st;
  if (s->n > 0 && (bad_ptr(s->means) || bad_ptr(s->log_scales) || bad_ptr(s->quats) || bad_ptr(s->opacity_logits)))
    return fail(ctx, GS_ERR_INVALID_ARG, "a geometry array is NULL or misaligned");
  return GS_OK;
}

// ---- workspace layout -------------------------------------------------------------------------
size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct Carver {
  char *base;
  size_t used;
  template <class T>
  T *take(size_t count) {
    T *p = reinterpret_cast<T *>(base + used);
    used += align_up(count * sizeof(T));
    return p;
  }
};

struct FwdWorkspace {
  uint32_t *sorted_depth, *tmp_keys, *tmp_vals;          // [n]
  uint32_t *block_sums;                                  // cell records per 256 depth-sorted Gaussians
  uint32_t *rec_keys, *rec_vals, *tmp_rkeys, *tmp_rvals; // [pair_capacity]: cell records (never more than instances, save for
                                                         // slivers that reach a cell's rows but none of its tiles)
  uint32_t *cell_ranges;                                 // [cells, 2]
  CellScratch cells;
  unsigned long long *rec_total;                         // number of records, written by the emission
  void *sort_table;
  size_t bytes;
};

FwdWorkspace carve_fwd(void *ws, int64_t n, int64_t cap, int width, int height) {
  Carver c{static_cast<char *>(ws), 0};
  FwdWorkspace w;
  const size_t nn = (size_t)(n > 0 ? n : 1), cc = (size_t)(cap > 0 ? cap : 1);
  const int gx = (width + GS_TILE - 1) / GS_TILE, gy = (height + GS_TILE - 1) / GS_TILE;
  const int cells = ((gx + 3) / 4) * ((gy + 3) / 4);
  const size_t chunks = (size_t)max_chunks((int64_t)cc, cells);
  w.sorted_depth = c.take<uint32_t>(nn);
  w.tmp_keys = c.take<uint32_t>(nn);
  w.tmp_vals = c.take<uint32_t>(nn);
  w.block_sums = reinterpret_cast<uint32_t *>(c.take<char>(scan_scratch_bytes((int64_t)nn)));
  w.rec_keys = c.take<uint32_t>(cc);
  w.rec_vals = c.take<uint32_t>(cc);
  w.tmp_rkeys = c.take<uint32_t>(cc);
  w.tmp_rvals = c.take<uint32_t>(cc);
  w.cell_ranges = c.take<uint32_t>((size_t)cells * 2);
  w.cells.chunk_first = c.take<uint32_t>((size_t)cells + 1);
  w.cells.chunk_counts = c.take<uint32_t>(chunks * 16);
  w.cells.chunk_bases = c.take<uint32_t>(chunks * 16);
  w.cells.tile_counts = c.take<uint32_t>((size_t)gx * gy);
  w.cells.tile_starts = c.take<uint32_t>((size_t)gx * gy);
  w.rec_total = c.take<unsigned long long>(1);
  w.sort_table = c.take<char>(sort_scratch_bytes((int64_t)(nn > cc ? nn : cc)));
  w.bytes = c.used;
  return w;
}

// Backward scratch: the 2D gradients [n,12], then (used by the separate-pass path only) directions, dL/dcolor and
// dL/dd as [n,3] each, then the flags of the Gaussians that received a gradient.
struct BwdWorkspace { float *g2d, *dirs, *g_color, *g_dirs; uint32_t *flags; size_t bytes; };
BwdWorkspace carve_bwd(void *ws, int64_t n) {
  Carver c{static_cast<char *>(ws), 0};
  const size_t nn = (size_t)(n > 0 ? n : 1);
  BwdWorkspace w;
  w.g2d = c.take<float>(nn * 12);
  w.dirs = c.take<float>(nn * 3);
  w.g_color = c.take<float>(nn * 3);
  w.g_dirs = c.take<float>(nn * 3);
  w.flags = c.take<uint32_t>((nn + 31) / 32);     // one bit per Gaussian: it received a gradient
  w.bytes = c.used;
  return w;
}
size_t bwd_bytes(int64_t n) { return carve_bwd(nullptr, n).bytes; }

int id_bits(int count) {
  int bits = 1;
  while ((1 << bits) < count) ++bits;
  return bits;
}

}  // namespace

extern "C" {

GsStatus gs_create(int device, GsContext **out) {
  if (!out) return GS_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return GS_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return GS_ERR_CUDA;
  GsContext *ctx = new (std::nothrow) GsContext();
  if (!ctx) return GS_ERR_INTERNAL;
  ctx->device = device;
  ctx->num_sms = 148;
  cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, device);
  ctx->error[0] = 0;
  ctx->d_counter = nullptr; ctx->h_counter = nullptr; ctx->d_w_partials = nullptr;
  ctx->profiling = false;
  ctx->decoder_engine = GS_ENGINE_AUTO;
  if (cudaMalloc(&ctx->d_counter, 8 * sizeof(unsigned long long)) != cudaSuccess ||
      cudaMemset(ctx->d_counter, 0, 8 * sizeof(unsigned long long)) != cudaSuccess ||
      cudaMallocHost(&ctx->h_counter, 8 * sizeof(unsigned long long)) != cudaSuccess ||
      cudaMalloc(&ctx->d_w_partials, sizeof(float) * std::max((size_t)kWgradBlocks * GS_MLP_WEIGHTS, variant_partials_floats())) != cudaSuccess) {
    gs_destroy(ctx);
    return GS_ERR_CUDA;
  }
  *out = ctx;
  return GS_OK;
}

void gs_destroy(GsContext *ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  if (ctx->d_counter) cudaFree(ctx->d_counter);
  if (ctx->h_counter) cudaFreeHost(ctx->h_counter);
  if (ctx->d_w_partials) cudaFree(ctx->d_w_partials);
  for (StageRecord &r : ctx->records) { cudaEventDestroy(r.begin); cudaEventDestroy(r.end); }
  for (cudaEvent_t e : ctx->free_events) cudaEventDestroy(e);
  delete ctx;
}

const char *gs_last_error(const GsContext *ctx) { return ctx ? ctx->error : "no context"; }

size_t gs_workspace_bytes(int64_t n, int32_t width, int32_t height, int64_t pair_capacity) {
  if (n < 0 || width <= 0 || height <= 0 || pair_capacity < 0) return 0;
  const size_t f = carve_fwd(nullptr, n, pair_capacity, width, height).bytes, b = bwd_bytes(n);
  return f > b ? f : b;
}

namespace {
GsStatus preprocess_impl(GsContext *ctx, const GsScene *scene, const GsCamera *cam, GsProjected *out,
                         int64_t *num_pairs_host, void *stream) {
  GsStatus st = scene_ok(ctx, scene);
  if (st != GS_OK) return st;
  if (!camera_ok(cam)) return fail(ctx, GS_ERR_INVALID_ARG, "bad camera (size, focal length, or more than 65536 cells of 64 x 64 pixels, e.g. beyond 16384 x 16384)");
  if (!out) return fail(ctx, GS_ERR_INVALID_ARG, "out is NULL");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  // the counter is cleared even for an empty scene: a device-counted forward reads it
  if ((st = check_cuda(ctx, cudaMemsetAsync(ctx->d_counter, 0, sizeof(unsigned long long), s), "memset")) != GS_OK) return st;
  if (scene->n == 0) return GS_OK;
  if (bad_ptr(out->mean2d) || bad_ptr(out->conic_opacity) || bad_ptr(out->color) || bad_ptr(out->depth_key) ||
      bad_ptr(out->rect) || bad_ptr(out->tiles_touched) || bad_ptr(out->cell_count) || bad_ptr(out->cell_records) ||
      (out->extent && !aligned16(out->extent)))
    return fail(ctx, GS_ERR_INVALID_ARG, "a GsProjected buffer is NULL or misaligned");
  PreprocessArgs a;
  a.n = scene->n;
  a.means = scene->means; a.log_scales = scene->log_scales; a.quats = scene->quats; a.logits = scene->opacity_logits;
  a.base_color = scene->base_color; a.sh_rest = scene->app == GS_APP_SV ? scene->sv_sites : scene->sh_rest;
  a.features = reinterpret_cast<const __half *>(scene->features);
  a.weights = reinterpret_cast<const __half *>(scene->mlp_weights);
  a.deg = scene->active_degree; a.act = scene->color_activation;
  a.mean2d = out->mean2d; a.conic_opacity = out->conic_opacity; a.color = out->color; a.extent = out->extent;
  a.depth_key = out->depth_key; a.rect = out->rect; a.tiles_touched = out->tiles_touched;
  a.cell_count = out->cell_count; a.cell_records = out->cell_records;
  a.pair_counter = ctx->d_counter;
  {
    StageTimer t(ctx, GS_STAGE_PREPROCESS_FWD, s);
    t.done(launch_preprocess_fwd(unfused(scene) ? kAppExternal : kernel_app(scene), a, make_cam(cam), s));
  }
  if (unfused(scene)) {   // directions sit in out->color: decode them in place, visible Gaussians only
    AppearanceArgs ap = appearance_args(ctx, scene);
    ap.dirs = out->color; ap.color = out->color; ap.mask = out->tiles_touched;
    StageTimer t(ctx, GS_STAGE_APPEARANCE_FWD, s);
    t.done(run_appearance_fwd(scene, ap, s));
  }
  if ((st = check_cuda(ctx, cudaGetLastError(), "preprocess launch")) != GS_OK) return st;
  if (!num_pairs_host) return GS_OK;
  if ((st = check_cuda(ctx, cudaMemcpyAsync(ctx->h_counter, ctx->d_counter, sizeof(unsigned long long),
                                            cudaMemcpyDeviceToHost, s), "pair count copy")) != GS_OK) return st;
  if ((st = check_cuda(ctx, cudaStreamSynchronize(s), "preprocess")) != GS_OK) return st;
  *num_pairs_host = (int64_t)*ctx->h_counter;
  return GS_OK;
}
}  // namespace

GsStatus gs_preprocess(GsContext *ctx, const GsScene *scene, const GsCamera *cam, GsProjected *out,
                       int64_t *num_pairs_host, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!num_pairs_host) return fail(ctx, GS_ERR_INVALID_ARG, "num_pairs_host is NULL");
  *num_pairs_host = 0;
  return preprocess_impl(ctx, scene, cam, out, num_pairs_host, stream);
}

GsStatus gs_preprocess_async(GsContext *ctx, const GsScene *scene, const GsCamera *cam, GsProjected *out, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  return preprocess_impl(ctx, scene, cam, out, nullptr, stream);
}

GsStatus gs_async_status(GsContext *ctx, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  GsStatus st;
  if ((st = check_cuda(ctx, cudaMemcpyAsync(ctx->h_counter + 2, ctx->d_counter + 2, 2 * sizeof(unsigned long long),
                                            cudaMemcpyDeviceToHost, s), "status copy")) != GS_OK) return st;
  if ((st = check_cuda(ctx, cudaMemsetAsync(ctx->d_counter + 2, 0, 2 * sizeof(unsigned long long), s), "status reset")) != GS_OK) return st;
  if ((st = check_cuda(ctx, cudaStreamSynchronize(s), "status")) != GS_OK) return st;
  if (ctx->h_counter[3] != 0)
    return fail(ctx, GS_ERR_INTERNAL, "a bounded wait on a bulk copy ran out in an appearance kernel: its results are incomplete");
  if (ctx->h_counter[2] != 0)
    return fail(ctx, GS_ERR_CAPACITY, "a device-counted gs_render_forward had more instances than pair_capacity: that view's lists were cut off");
  return GS_OK;
}

GsStatus gs_render_forward(GsContext *ctx, int64_t n, const GsProjected *proj, const GsCamera *cam,
                           int64_t num_pairs, int64_t pair_capacity, GsBinning *bin, float *image,
                           float *final_T, uint32_t *n_contrib, void *workspace, size_t workspace_bytes,
                           void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  const bool on_device = num_pairs == GS_PAIRS_ON_DEVICE;   // the count of the context's last gs_preprocess(_async)
  const unsigned long long *count_dev = on_device ? ctx->d_counter : nullptr;
  if (on_device) num_pairs = pair_capacity;
  if (n < 0 || num_pairs < 0 || pair_capacity < 0) return fail(ctx, GS_ERR_INVALID_ARG, "negative size");
  if (!camera_ok(cam)) return fail(ctx, GS_ERR_INVALID_ARG, "bad camera");
  if (!proj || !bin) return fail(ctx, GS_ERR_INVALID_ARG, "proj / bin is NULL");
  if (bad_ptr(image) || bad_ptr(final_T) || bad_ptr(n_contrib) || bad_ptr(bin->tile_ranges) || bad_ptr(bin->tile_order))
    return fail(ctx, GS_ERR_INVALID_ARG, "an output buffer is NULL or misaligned");
  if (num_pairs > pair_capacity) return fail(ctx, GS_ERR_CAPACITY, "num_pairs exceeds pair_capacity");
  if (num_pairs >= ((int64_t)1 << 32)) return fail(ctx, GS_ERR_CAPACITY, "more than 2^32 - 1 instances");
  if (workspace_bytes < gs_workspace_bytes(n, cam->width, cam->height, pair_capacity) || bad_ptr(workspace))
    return fail(ctx, GS_ERR_CAPACITY, "workspace is NULL, misaligned or smaller than gs_workspace_bytes()");
  if (n > 0 && (bad_ptr(proj->mean2d) || bad_ptr(proj->conic_opacity) || bad_ptr(proj->color) ||
                bad_ptr(proj->depth_key) || bad_ptr(proj->rect) || bad_ptr(proj->tiles_touched) ||
                bad_ptr(bin->depth_order)))
    return fail(ctx, GS_ERR_INVALID_ARG, "a per-Gaussian buffer is NULL or misaligned");
  if (num_pairs > 0 && (bad_ptr(bin->sorted_tiles) || bad_ptr(bin->sorted_vals)))
    return fail(ctx, GS_ERR_INVALID_ARG, "an instance buffer is NULL or misaligned");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  const CamDev cd = make_cam(cam);
  const int num_tiles = cd.gx * cd.gy;
  const FwdWorkspace w = carve_fwd(workspace, n, pair_capacity, cam->width, cam->height);
  const bool sorted = n > 0 && num_pairs > 0;
  if (sorted) {
    uint32_t *overflow = reinterpret_cast<uint32_t *>(ctx->d_counter + 2);
    // stage 1: Gaussians by depth key (stable => ties keep the index order); the last pass also leaves the cell records
    // per 256 sorted Gaussians, from which their emission takes its offsets
    {
      StageTimer t(ctx, GS_STAGE_DEPTH_SORT, s);
      const SortEpilogue ep = {proj->cell_count, ~kCellBig, w.block_sums, num_scan_blocks(n), nullptr, 0, 0, nullptr};
      t.done(launch_radix_sort(proj->depth_key, nullptr, w.sorted_depth, bin->depth_order, w.tmp_keys, w.tmp_vals,
                               n, nullptr, 0, 32, 8, w.sort_table, &ep, s));
    }
    // stage 2: one record per (Gaussian, cell of 4 x 4 tiles) in depth order, then a stable sort by cell id alone,
    // whose last pass finds where every cell's records begin and end
    {
      StageTimer t(ctx, GS_STAGE_KEYGEN, s);
      t.done(launch_emit_records(bin->depth_order, proj->cell_count, proj->cell_records, proj->rect, proj->mean2d,
                                 proj->conic_opacity, w.block_sums, w.rec_keys, w.rec_vals, w.rec_total, overflow, n, cd.cgx,
                                 cd.W, cd.H, pair_capacity, s));
    }
    const int num_cells = cd.cgx * cd.cgy;
    // two buffers serve the passes: an odd number of passes ends in the other one, an even number back in the first
    const int cell_bits = id_bits(num_cells);
    constexpr int kCellDigit = 9;   // up to 512 cells (2048 x 1024 pixels) sort in one pass
    const bool odd = (radix_passes(cell_bits, kCellDigit) & 1) != 0;
    uint32_t *sorted_rkeys = odd ? w.tmp_rkeys : w.rec_keys, *sorted_rvals = odd ? w.tmp_rvals : w.rec_vals;
    {
      StageTimer t(ctx, GS_STAGE_TILE_SORT, s);
      const SortEpilogue ep = {nullptr, 0u, nullptr, 0, w.cell_ranges, num_cells, 16, nullptr};
      // the count lives on the device; its host-side bound: a record holds at least one instance
      t.done(launch_radix_sort(w.rec_keys, w.rec_vals, sorted_rkeys, sorted_rvals, odd ? w.rec_keys : w.tmp_rkeys,
                               odd ? w.rec_vals : w.tmp_rvals, num_pairs, w.rec_total, 16, cell_bits, kCellDigit, w.sort_table, &ep, s));
    }
    // stage 3: the records of every cell, still in depth order, expanded into the lists of its 16 tiles
    {
      StageTimer t(ctx, GS_STAGE_TILE_RANGES, s);
      if (on_device)   // more instances than the capacity: the lists are cut off, the host is told
        launch_flag_if_greater(count_dev, (unsigned long long)pair_capacity, overflow, s);
      t.done(launch_expand(sorted_rkeys, sorted_rvals, w.cell_ranges, w.cells, num_pairs, pair_capacity, cd.gx, cd.gy, cd.cgx,
                           cd.cgy, bin->sorted_vals, bin->tile_ranges, bin->tile_order, s));
    }
  } else {
    StageTimer t(ctx, GS_STAGE_TILE_RANGES, s);
    t.done(launch_empty_binning(bin->tile_ranges, bin->tile_order, num_tiles, s));
  }
  {
    StageTimer t(ctx, GS_STAGE_BLEND_FWD, s);
    t.done(launch_blend_fwd(cd, bin->tile_ranges, bin->tile_order, bin->sorted_vals, proj->mean2d, proj->conic_opacity, proj->color,
                            num_pairs > 0 ? bin->sorted_tiles : nullptr, image, final_T, n_contrib, s));
  }
  return check_cuda(ctx, cudaGetLastError(), "render_forward launch");
}

GsStatus gs_render_backward(GsContext *ctx, const GsScene *scene, const GsCamera *cam, const GsProjected *proj,
                            const GsBinning *bin, int64_t num_pairs, const float *final_T,
                            const uint32_t *n_contrib, const float *dL_dimage, GsGrads *grads, void *workspace,
                            size_t workspace_bytes, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  GsStatus st = scene_ok(ctx, scene);
  if (st != GS_OK) return st;
  if (!camera_ok(cam)) return fail(ctx, GS_ERR_INVALID_ARG, "bad camera");
  if (!proj || !bin || !grads) return fail(ctx, GS_ERR_INVALID_ARG, "proj / bin / grads is NULL");
  if (num_pairs == GS_PAIRS_ON_DEVICE) num_pairs = 1;   // unknown here; the tile ranges bound every list
  if (bad_ptr(final_T) || bad_ptr(n_contrib) || bad_ptr(dL_dimage) || bad_ptr(bin->tile_ranges) || bad_ptr(bin->tile_order))
    return fail(ctx, GS_ERR_INVALID_ARG, "an image-sized buffer is NULL or misaligned");
  const int64_t n = scene->n;
  if (scene->app == GS_APP_NEURAL && bad_ptr(grads->mlp_weights))
    return fail(ctx, GS_ERR_INVALID_ARG, "grads->mlp_weights is NULL or misaligned");
  if (n > 0) {
    if (bad_ptr(grads->means) || bad_ptr(grads->log_scales) || bad_ptr(grads->quats) ||
        bad_ptr(grads->opacity_logits) || bad_ptr(grads->base_color))
      return fail(ctx, GS_ERR_INVALID_ARG, "a gradient buffer is NULL or misaligned");
    if (scene->app == GS_APP_SH && bad_ptr(grads->sh_rest)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->sh_rest is NULL or misaligned");
    if (scene->app == GS_APP_SV && bad_ptr(grads->sv_sites)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->sv_sites is NULL or misaligned");
    if (scene->app == GS_APP_NEURAL && bad_ptr(grads->features)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->features is NULL or misaligned");
    if (bad_ptr(proj->mean2d) || bad_ptr(proj->conic_opacity) || bad_ptr(proj->color) || bad_ptr(proj->rect))
      return fail(ctx, GS_ERR_INVALID_ARG, "a GsProjected buffer is NULL or misaligned");
  }
  if (num_pairs > 0 && bad_ptr(bin->sorted_vals)) return fail(ctx, GS_ERR_INVALID_ARG, "sorted_vals is NULL or misaligned");
  if (workspace_bytes < bwd_bytes(n) || bad_ptr(workspace))
    return fail(ctx, GS_ERR_CAPACITY, "workspace is NULL, misaligned or too small");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  const CamDev cd = make_cam(cam);
  const BwdWorkspace bw = carve_bwd(workspace, n);
  float *g2d = bw.g2d;
  const bool ext = unfused(scene);
  if (ext && n > 0 && bad_ptr(proj->tiles_touched)) return fail(ctx, GS_ERR_INVALID_ARG, "proj->tiles_touched is NULL or misaligned");
  if (n > 0) {
    if ((st = check_cuda(ctx, cudaMemsetAsync(g2d, 0, (size_t)n * 12 * sizeof(float), s), "memset")) != GS_OK) return st;
    if (num_pairs > 0) {
      StageTimer t(ctx, GS_STAGE_BLEND_BWD, s);
      t.done(launch_blend_bwd(cd, bin->tile_ranges, bin->tile_order, bin->sorted_vals, proj->mean2d, proj->conic_opacity, proj->color,
                              final_T, n_contrib, dL_dimage, g2d, s));
    }
  }
  PreprocessBwdArgs a;
  a.n = n;
  a.means = scene->means; a.log_scales = scene->log_scales; a.quats = scene->quats; a.logits = scene->opacity_logits;
  a.base_color = scene->base_color; a.sh_rest = scene->app == GS_APP_SV ? scene->sv_sites : scene->sh_rest;
  a.features = reinterpret_cast<const __half *>(scene->features);
  a.weights = reinterpret_cast<const __half *>(scene->mlp_weights);
  a.deg = scene->active_degree; a.act = scene->color_activation;
  a.rect = proj->rect; a.g2d = g2d;
  a.g_means = grads->means; a.g_log_scales = grads->log_scales; a.g_quats = grads->quats;
  a.g_logits = grads->opacity_logits; a.g_base = grads->base_color;
  a.g_sh_rest = scene->app == GS_APP_SV ? grads->sv_sites : grads->sh_rest;
  a.g_features = grads->features; a.w_partials = ctx->d_w_partials; a.g_weights = grads->mlp_weights;
  a.gd_in = bw.g_dirs;
  a.flags = bw.flags;
  a.nfeat = scene->app == GS_APP_NEURAL ? decoder_arch(scene).nfeat : 8;
  a.timeout = ctx->d_counter + 3;
  if (n == 0 && scene->app == GS_APP_NEURAL) {
    const DecoderArch d = decoder_arch(scene);
    return check_cuda(ctx, cudaMemsetAsync(grads->mlp_weights, 0, sizeof(float) * variant_num_weights(d.hidden, d.layers), s), "memset");
  }
  bool flags_ready = false;
  if (ext && n > 0) {   // the appearance backward as a pass of its own, through dense arrays in the workspace
    AppearanceArgs ap = appearance_args(ctx, scene);
    ap.dirs = bw.dirs; ap.g_color = bw.g_color; ap.mask = proj->tiles_touched;
    ap.g_base = grads->base_color; ap.g_sh_rest = scene->app == GS_APP_SV ? grads->sv_sites : grads->sh_rest;
    ap.g_features = grads->features; ap.g_dirs = bw.g_dirs;
    ap.w_partials = ctx->d_w_partials; ap.g_weights = grads->mlp_weights;
    // A decoder variant on the tcgen05 kernels works on the Gaussians that received a gradient only: the flag bits
    // (and the zero rows of everyone else) are taken first, and serve the projection backward below as well.
    flags_ready = scene->app == GS_APP_NEURAL && !default_decoder(scene) && ctx->decoder_engine != GS_ENGINE_WARP_MMA && scene->active_degree > 0;
    StageTimer t(ctx, GS_STAGE_APPEARANCE_BWD, s);
    int launches = 0;
    if (flags_ready) {   // directions and dL/dcolor are taken from the means and the 2D gradient rows in the kernel itself
      launches = launch_bwd_flags(a, true, s);
      ap.flags = bw.flags;
      ap.means = scene->means; ap.g2d = g2d;
      ap.oc[0] = cd.oc[0]; ap.oc[1] = cd.oc[1]; ap.oc[2] = cd.oc[2];
    } else {
      launches = launch_unfused_prepare(n, scene->means, cd, g2d, proj->tiles_touched, bw.dirs, bw.g_color, s);
    }
    t.done(launches + run_appearance_bwd(scene, ap, s));
  }
  {
    StageTimer t(ctx, GS_STAGE_PREPROCESS_BWD, s);
    t.done(launch_preprocess_bwd(ext ? kAppExternal : kernel_app(scene), a, cd, s, flags_ready));
  }
  return check_cuda(ctx, cudaGetLastError(), "render_backward launch");
}

GsStatus gs_appearance_forward(GsContext *ctx, const GsScene *scene, const float *dirs, float *color, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!scene) return fail(ctx, GS_ERR_INVALID_ARG, "scene is NULL");
  GsStatus st = scene_appearance_ok(ctx, scene);
  if (st != GS_OK) return st;
  if (scene->n == 0) return GS_OK;
  if (bad_ptr(dirs) || bad_ptr(color)) return fail(ctx, GS_ERR_INVALID_ARG, "dirs / color is NULL or misaligned");
  cudaSetDevice(ctx->device);
  AppearanceArgs a = appearance_args(ctx, scene);
  a.dirs = dirs;
  a.color = color;
  {
    StageTimer t(ctx, GS_STAGE_APPEARANCE_FWD, static_cast<cudaStream_t>(stream));
    t.done(run_appearance_fwd(scene, a, static_cast<cudaStream_t>(stream)));
  }
  return check_cuda(ctx, cudaGetLastError(), "appearance_forward launch");
}

GsStatus gs_appearance_backward(GsContext *ctx, const GsScene *scene, const float *dirs, const float *dL_dcolor,
                                GsGrads *grads, float *dL_ddirs, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!scene || !grads) return fail(ctx, GS_ERR_INVALID_ARG, "scene / grads is NULL");
  GsStatus st = scene_appearance_ok(ctx, scene);
  if (st != GS_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  if (scene->app == GS_APP_NEURAL && bad_ptr(grads->mlp_weights))
    return fail(ctx, GS_ERR_INVALID_ARG, "grads->mlp_weights is NULL or misaligned");
  if (scene->n == 0) {
    if (scene->app == GS_APP_NEURAL) {
      const DecoderArch d = decoder_arch(scene);
      return check_cuda(ctx, cudaMemsetAsync(grads->mlp_weights, 0, sizeof(float) * variant_num_weights(d.hidden, d.layers), s), "memset");
    }
    return GS_OK;
  }
  if (bad_ptr(dirs) || bad_ptr(dL_dcolor) || bad_ptr(dL_ddirs) || bad_ptr(grads->base_color))
    return fail(ctx, GS_ERR_INVALID_ARG, "dirs / dL_dcolor / dL_ddirs / grads->base_color is NULL or misaligned");
  if (scene->app == GS_APP_SH && bad_ptr(grads->sh_rest)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->sh_rest is NULL or misaligned");
  if (scene->app == GS_APP_SV && bad_ptr(grads->sv_sites)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->sv_sites is NULL or misaligned");
  if (scene->app == GS_APP_NEURAL && bad_ptr(grads->features)) return fail(ctx, GS_ERR_INVALID_ARG, "grads->features is NULL or misaligned");
  AppearanceArgs a = appearance_args(ctx, scene);
  a.dirs = dirs;
  a.g_color = dL_dcolor;
  a.g_base = grads->base_color; a.g_sh_rest = scene->app == GS_APP_SV ? grads->sv_sites : grads->sh_rest;
  a.g_features = grads->features; a.g_dirs = dL_ddirs;
  a.w_partials = ctx->d_w_partials; a.g_weights = grads->mlp_weights;
  {
    StageTimer t(ctx, GS_STAGE_APPEARANCE_BWD, s);
    t.done(run_appearance_bwd(scene, a, s));
  }
  return check_cuda(ctx, cudaGetLastError(), "appearance_backward launch");
}

GsStatus gs_profile_blend_counts(GsContext *ctx, const GsProjected *proj, const GsBinning *bin, const GsCamera *cam,
                                 int64_t *counts_host, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!proj || !bin || !counts_host || !camera_ok(cam)) return fail(ctx, GS_ERR_INVALID_ARG, "bad argument");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  GsStatus st;
  if ((st = check_cuda(ctx, cudaMemsetAsync(ctx->d_counter + 4, 0, 4 * sizeof(unsigned long long), s), "memset")) != GS_OK) return st;
  launch_blend_count(make_cam(cam), bin->tile_ranges, bin->sorted_vals, proj->mean2d, proj->conic_opacity, proj->color,
                     ctx->d_counter + 4, s);
  if ((st = check_cuda(ctx, cudaMemcpyAsync(ctx->h_counter + 4, ctx->d_counter + 4, 4 * sizeof(unsigned long long),
                                            cudaMemcpyDeviceToHost, s), "count copy")) != GS_OK) return st;
  if ((st = check_cuda(ctx, cudaStreamSynchronize(s), "blend counts")) != GS_OK) return st;
  for (int k = 0; k < 4; ++k) counts_host[k] = (int64_t)ctx->h_counter[4 + k];
  return GS_OK;
}

GsStatus gs_adam_step(GsContext *ctx, const GsAdamTensor *tensors, int32_t num_tensors, int64_t step, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (num_tensors < 0 || num_tensors > GS_ADAM_MAX_TENSORS || (num_tensors > 0 && !tensors))
    return fail(ctx, GS_ERR_INVALID_ARG, "num_tensors must be 0..8 and tensors non-NULL");
  if (step < 1) return fail(ctx, GS_ERR_INVALID_ARG, "step counts from 1");
  for (int i = 0; i < num_tensors; ++i) {
    const GsAdamTensor &t = tensors[i];
    if (t.rows < 0 || t.cols < 1 || t.cols > GS_ADAM_MAX_COLS) return fail(ctx, GS_ERR_INVALID_ARG, "rows < 0 or cols outside 1..64");
    if (t.rows == 0) continue;
    if (!t.lr) return fail(ctx, GS_ERR_INVALID_ARG, "lr is NULL");
    if (bad_ptr(t.param) || bad_ptr(t.grad) || bad_ptr(t.exp_avg) || bad_ptr(t.exp_avg_sq) ||
        (t.half_copy && (reinterpret_cast<uintptr_t>(t.half_copy) & 7u)))
      return fail(ctx, GS_ERR_INVALID_ARG, "an Adam tensor pointer is NULL or misaligned");
    if (!(t.beta1 >= 0.f && t.beta1 < 1.f && t.beta2 >= 0.f && t.beta2 < 1.f) || !(t.eps >= 0.f))
      return fail(ctx, GS_ERR_INVALID_ARG, "betas must lie in [0, 1) and eps be >= 0");
    if ((uint64_t)t.rows * (uint64_t)t.cols >= (1ull << 32)) return fail(ctx, GS_ERR_CAPACITY, "an Adam tensor has 2^32 elements or more");
    if (t.num_more_grads < 0 || t.num_more_grads > GS_ADAM_MAX_MORE_GRADS || (t.num_more_grads > 0 && !t.more_grads))
      return fail(ctx, GS_ERR_INVALID_ARG, "num_more_grads outside 0..7 or more_grads is NULL");
    for (int k = 0; k < t.num_more_grads; ++k)
      if (bad_ptr(t.more_grads[k])) return fail(ctx, GS_ERR_INVALID_ARG, "a further gradient pointer is NULL or misaligned");
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  {
    StageTimer t(ctx, GS_STAGE_ADAM, s);
    t.done(launch_adam(tensors, num_tensors, step, ctx->num_sms, s));
  }
  return check_cuda(ctx, cudaGetLastError(), "adam launch");
}

GsStatus gs_neural_fold(GsContext *ctx, const GsScene *scene, uint16_t *preact, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!scene || scene->n < 0) return fail(ctx, GS_ERR_INVALID_ARG, "scene is NULL or n < 0");
  if (scene->app != GS_APP_NEURAL) return fail(ctx, GS_ERR_UNSUPPORTED, "the fold exists for the neural model only");
  if (!default_decoder(scene)) return fail(ctx, GS_ERR_UNSUPPORTED, "the fold is built for the 16 / 2 / 8 decoder only");
  if (scene->n == 0) return GS_OK;
  if (bad_ptr(scene->features) || bad_ptr(scene->mlp_weights) || bad_ptr(preact))
    return fail(ctx, GS_ERR_INVALID_ARG, "features, mlp_weights or preact is NULL or misaligned");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  {
    StageTimer t(ctx, GS_STAGE_PREPASS, s);
    t.done(launch_neural_fold(scene->n, reinterpret_cast<const __half *>(scene->features),
                              reinterpret_cast<const __half *>(scene->mlp_weights), reinterpret_cast<__half *>(preact), s));
  }
  return check_cuda(ctx, cudaGetLastError(), "neural fold launch");
}

GsStatus gs_neural_prepass(GsContext *ctx, const GsScene *scene, const uint16_t *preact, const GsCamera *cam,
                           uint8_t *rgba, float *color, void *stream) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (!scene || scene->n < 0 || !cam) return fail(ctx, GS_ERR_INVALID_ARG, "scene or cam is NULL, or n < 0");
  if (scene->app != GS_APP_NEURAL) return fail(ctx, GS_ERR_UNSUPPORTED, "the prepass exists for the neural model only");
  if (!default_decoder(scene)) return fail(ctx, GS_ERR_UNSUPPORTED, "the prepass is built for the 16 / 2 / 8 decoder only");
  if (scene->active_degree < 0 || scene->active_degree > 3) return fail(ctx, GS_ERR_INVALID_ARG, "active_degree outside 0..3");
  if (scene->color_activation < GS_ACT_RELU || scene->color_activation > GS_ACT_HARD_SIGMOID)
    return fail(ctx, GS_ERR_INVALID_ARG, "unknown colour activation");
  if (scene->n == 0) return GS_OK;
  if (bad_ptr(scene->means) || bad_ptr(scene->opacity_logits) || bad_ptr(scene->base_color) || bad_ptr(scene->mlp_weights) ||
      bad_ptr(preact) || !rgba || (reinterpret_cast<uintptr_t>(rgba) & 3u) || (color && !aligned16(color)))
    return fail(ctx, GS_ERR_INVALID_ARG, "a prepass pointer is NULL or misaligned");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaSetDevice(ctx->device);
  const CamDev cd = make_cam(cam);
  {
    StageTimer t(ctx, GS_STAGE_PREPASS, s);
    t.done(launch_neural_prepass(scene->n, scene->active_degree, scene->color_activation, scene->means, scene->opacity_logits, scene->base_color,
                                 reinterpret_cast<const __half *>(preact), reinterpret_cast<const __half *>(scene->mlp_weights),
                                 cd.oc, rgba, color, s));
  }
  return check_cuda(ctx, cudaGetLastError(), "neural prepass launch");
}

GsStatus gs_profile_enable(GsContext *ctx, int enable) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  ctx->profiling = enable != 0;
  return GS_OK;
}

GsStatus gs_set_decoder_engine(GsContext *ctx, int engine) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  if (engine != GS_ENGINE_WARP_MMA && engine != GS_ENGINE_TCGEN05 && engine != GS_ENGINE_AUTO) return fail(ctx, GS_ERR_INVALID_ARG, "unknown decoder engine");
  ctx->decoder_engine = engine;
  return GS_OK;
}

GsStatus gs_profile_collect(GsContext *ctx, double *ms, int64_t *launches) {
  if (!ctx) return GS_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  GsStatus st = GS_OK;
  for (StageRecord &r : ctx->records) {
    float t = 0.f;
    cudaError_t e = cudaEventSynchronize(r.end);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, r.begin, r.end);
    if (e != cudaSuccess) st = check_cuda(ctx, e, "profile collect");
    else {
      if (ms) ms[r.stage] += (double)t;
      if (launches) launches[r.stage] += r.launches;
    }
    ctx->free_events.push_back(r.begin);
    ctx->free_events.push_back(r.end);
  }
  ctx->records.clear();
  return st;
}

}  // extern "C"
