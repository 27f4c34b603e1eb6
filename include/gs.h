/*
 * gs.h - C ABI of the B200 (sm_100a) differentiable Gaussian-splatting step with fused
 * view-dependent appearance.
 *
 * The library implements one training-step hot path: per-Gaussian preprocess (projection to the
 * image plane, 16x16 tile overlap, view-dependent colour), tile/depth ordering, per-tile
 * front-to-back alpha blending, and the backward pass to every per-Gaussian parameter and to
 * the shared decoder weights (Sec. 3.1 "Appearance Modelling in Gaussian Splatting", Sec. 4
 * "Neural View-Dependent Appearance" and its "CUDA Implementation" paragraph).
 *
 * Conventions
 *   - Every pointer in GsScene / GsProjected / GsBinning / GsGrads and every `float *` / `void *`
 *     argument is a DEVICE pointer owned by the caller, contiguous, 16-byte aligned, unless the
 *     comment says "host".  The structs themselves live in host memory.
 *   - The library allocates nothing per call.  Work is enqueued on the caller's stream
 *     (`stream` is a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - Outputs are overwritten, never accumulated into.
 *   - Every call returns a GsStatus; no exception, device trap or device assert crosses the
 *     boundary.  gs_last_error() gives a text for the last failure on that context.
 *   - Camera frame: +x right, +y down, +z forward; pixel (i, j) has its centre at (i+0.5, j+0.5).
 *   - Non-finite values in a Gaussian's inputs cull that Gaussian (defined behaviour).
 */
#ifndef GS_B200_H_
#define GS_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct GsContext GsContext;

typedef enum {
  GS_OK = 0,
  GS_ERR_INVALID_ARG = -1, /* NULL / misaligned pointer, n < 0, bad image size, bad degree ... */
  GS_ERR_CAPACITY = -2,    /* pair count exceeds pair_capacity or workspace too small          */
  GS_ERR_CUDA = -3,        /* a CUDA runtime call failed; see gs_last_error                    */
  GS_ERR_UNSUPPORTED = -4,
  GS_ERR_INTERNAL = -6
} GsStatus;

typedef enum {
  GS_APP_SH = 0,      /* spherical harmonics, degrees 1..3 (Eq. 1)                              */
  GS_APP_NEURAL = 1,  /* latent features + shared decoder (Eq. 5-7)                             */
  GS_APP_SV = 2       /* Spherical Voronoi: soft interpolation over seven sites (Eq. 3)         */
} GsAppearance;

enum {
  GS_TILE = 16,            /* tile edge in pixels (Sec. 3.1)                                    */
  GS_SV_SITES = 7,         /* Spherical Voronoi sites per Gaussian (App. B)                       */
  GS_SV_ROW = 49,          /* 7 sites x (colour a [3], unnormalised direction s [3], log-temperature) */
  GS_SH_REST = 45,         /* view-dependent SH coefficients per Gaussian, degrees 1..3, x RGB  */
  GS_NUM_FEATURES = 8,     /* F, latent features per Gaussian (Sec. 4)                          */
  GS_MLP_IN = 32,          /* D = 16 direction encodings + 16 feature encodings (Eq. 5)         */
  GS_MLP_HIDDEN = 16,
  GS_MLP_OUT = 3,
  GS_MLP_WEIGHTS = 816     /* 32*16 + 16*16 + 16*3, no biases (Sec. 4)                          */
};

/* Colour activation phi of Sec. 3.1, applied to x = c0 + A(d).  All four map 0 to (about) 0.5 with slope
 * (about) 1 there; the paper uses the first unless it says otherwise. */
typedef enum {
  GS_ACT_RELU = 0,         /* ReLU(x + 0.5), the standard one                                   */
  GS_ACT_SOFTPLUS = 1,     /* softplus(x + 0.5) with beta = 10                                  */
  GS_ACT_SIGMOID = 2,      /* sigmoid(4 x)                                                      */
  GS_ACT_HARD_SIGMOID = 3  /* clamp(x + 0.5, 0, 1)                                              */
} GsColorActivation;

typedef enum { GS_DECODER_SPLIT = 0, GS_DECODER_HALF = 1 } GsDecoderPrecision;

/* Pinhole camera (host struct). */
typedef struct {
  int32_t width, height;        /* pixels; at most 65535 tiles of 16 pixels per axis and 2^24
                                   tiles in all (GS_ERR_INVALID_ARG beyond)                    */
  float fx, fy, cx, cy;         /* intrinsics in pixel units                                   */
  float w2c[12];                /* row-major [R|t]: x_cam = R x_world + t                      */
  float near_plane, far_plane;  /* depth cull, typically 0.2 and 1e10                          */
  float background[3];          /* constant RGB composited behind everything                   */
} GsCamera;

/* The scene: per-Gaussian parameters plus the shared decoder (host struct of device pointers). */
typedef struct {
  int64_t n;                     /* number of Gaussians, >= 0 and < 2^31 (GS_ERR_CAPACITY)     */
  const float *means;            /* [n,3]                                                      */
  const float *log_scales;       /* [n,3]   scale = exp(log_scale)                             */
  const float *quats;            /* [n,4]   (w,x,y,z), normalised inside                       */
  const float *opacity_logits;   /* [n]     opacity = sigmoid(logit)                           */
  const float *base_color;       /* [n,3]   c0 of Eq. 2 (the constant Y0 is folded in)         */
  int32_t app;                   /* GsAppearance                                               */
  int32_t active_degree;         /* 0..3: direction bands in use (progressive schedule, Sec. 4);
                                    0 disables the view-dependent residual                     */
  const float *sh_rest;          /* SH only:     [n,15,3] bands 1..3, RGB innermost (Eq. 1)    */
  const uint16_t *features;      /* neural only: [n,8] IEEE fp16 bit patterns (Sec. 4)         */
  const uint16_t *mlp_weights;   /* neural only: [816] fp16: W1[16][32], W2[16][16], W3[3][16],
                                    each row-major (out, in); input order = 16 SH basis values
                                    of the direction, then (sin f_j, cos f_j) per feature
                                    (Eq. 5, Eq. 6 with k = 1)                                  */
  int32_t color_activation;      /* GsColorActivation: phi of c = phi(c0 + A(d)) (Sec. 3.1)    */
  const float *sv_sites;         /* SV only: [n,7,7] raw site parameters, per site (a_r, a_g, a_b, s_x,
                                    s_y, s_z, t): A(d) = sum_i softmax_i(-exp(t_i) |s_i/|s_i| - d|) a_i
                                    (Eq. 3 with the chord distance of App. B); any active_degree >= 1
                                    uses all seven sites, 0 disables the residual                  */
  int32_t mlp_hidden;            /* neural only: neurons per hidden layer, 16 or 32; 0 means 16   */
  int32_t mlp_layers;            /* neural only: hidden layers, 1..3; 0 means 2                   */
  int32_t num_features;          /* neural only: 8 (frequency encoded, Eq. 6) or 16 (fed to the decoder
                                    as they are, features then [n,16]); 0 means 8.  These three select a
                                    decoder of the architecture table (App. D): mlp_weights then holds
                                    W_1[hidden][32], (layers - 1) x [hidden][hidden], W_out[3][hidden],
                                    32 hidden + (layers - 1) hidden^2 + 3 hidden values.  Anything but
                                    the default 16 / 2 / 8 runs on plain fp32 kernels and, in the
                                    rendering step, always through the separate-pass path below;
                                    gs_neural_fold, gs_neural_prepass and
                                    gs_appearance_backward_noalloc return GS_ERR_UNSUPPORTED for it */
  int32_t separate_pass;         /* 0: appearance fused into the preprocess kernels (Sec. 4 "CUDA
                                    Implementation").  1: the unfused reference path of Sec. 4 / App. D
                                    "Fusion": gs_preprocess leaves the view directions of the visible
                                    Gaussians in GsProjected.color and a separate appearance pass turns
                                    them into colours in place; gs_render_backward runs the appearance
                                    backward as a pass of its own between the blend backward and the
                                    projection backward, exchanging directions, dL/dcolor and dL/dd
                                    through the workspace.  Same results up to rounding             */
  int32_t decoder_precision;     /* neural, default decoder only.  GS_DECODER_SPLIT (0): every product of
                                    the decoder takes its fp32 activation or gradient as two fp16 halves
                                    (fp32 accumulation), which keeps the results as accurate as fp32 FMAs:
                                    the mode every stated tolerance refers to.  GS_DECODER_HALF (1): plain
                                    fp16 operands with fp32 accumulation, the precision the paper runs its
                                    decoder in (Sec. 4 "CUDA Implementation"): about half the tensor-core
                                    work; colours then carry errors of the order of 1e-3                  */
} GsScene;

/* Per-Gaussian results of gs_preprocess (caller-allocated device buffers). */
typedef struct {
  float *mean2d;         /* [n,2]  projected centre in pixels                                  */
  float *conic_opacity;  /* [n,4]  (l11, l21, l22, opacity): the inverse 2D covariance ("conic") in
                                   Cholesky form, Q = L L^T with L = [[l11, 0], [l21, l22]], i.e.
                                   Q = [[l11^2, l11 l21], [l11 l21, l21^2 + l22^2]]                */
  float *color;          /* [n,3]  decoded view-dependent colour (Eq. 2)                       */
  uint32_t *depth_key;   /* [n]    bit pattern of the fp32 camera depth; 0xFFFFFFFF if culled  */
  uint16_t *rect;        /* [n,4]  tile rectangle (tx0, ty0, tx1, ty1), half open, bounding the
                                   alpha >= 1/255 footprint; all zero if the Gaussian touches no tile */
  uint32_t *tiles_touched; /* [n]  tiles inside rect that the alpha >= 1/255 ellipse really meets
                                   (= instances emitted for the Gaussian)                      */
  float *extent;         /* [n,4]  optional (may be NULL): (ex, ey, tau, 0): half-size in pixels of the
                                   box that bounds alpha >= 1/255 and tau = 2 ln(255 opacity);
                                   ex = ey = -1 if culled before the box test                  */
  /* The same footprint by cells of 4 x 4 tiles (64 x 64 pixels), for the binning of gs_render_forward: one
   * record per cell the footprint reaches, (cell id << 16) | 16-bit mask of the tiles it meets inside the
   * cell (bit 4 (ty % 4) + tx % 4; cell id = (ty / 4) * ceil(tiles_x / 4) + tx / 4), cells in row-major
   * order.  Opaque to the caller: allocate and pass on. */
  uint32_t *cell_count;    /* [n]    number of records; bit 31 set: more cells than 3 x 3, records not stored
                                     (gs_render_forward derives them again); 0 if the Gaussian touches no tile */
  uint32_t *cell_records;  /* [n,9]  the records of a Gaussian whose rectangle spans at most 3 x 3 cells      */
} GsProjected;

/* Tile binning produced by gs_render_forward (caller-allocated device buffers). */
typedef struct {
  uint32_t *depth_order;   /* [n]             Gaussian ids by (depth_key, id) ascending        */
  uint32_t *sorted_tiles;  /* [pair_capacity] tile id of each instance, ascending              */
  uint32_t *sorted_vals;   /* [pair_capacity] Gaussian id of each instance; inside a tile by
                                              (depth_key, id) ascending                        */
  uint32_t *tile_ranges;   /* [tiles,2]       [start,end) into the sorted lists, tiles =
                                              ceil(W/16)*ceil(H/16), row-major                 */
  uint32_t *tile_order;    /* [tiles]         tile ids by decreasing list length: the order in
                                              which the blend kernels start their tiles (affects
                                              scheduling only; ties in no particular order)    */
} GsBinning;

/* Gradients (caller-allocated device buffers, fp32, dense, exact zeros for culled Gaussians). */
typedef struct {
  float *means;           /* [n,3]                                                             */
  float *log_scales;      /* [n,3]                                                             */
  float *quats;           /* [n,4]  with respect to the un-normalised quaternion               */
  float *opacity_logits;  /* [n]                                                               */
  float *base_color;      /* [n,3]                                                             */
  float *sh_rest;         /* SH:     [n,15,3]                                                  */
  float *features;        /* neural: [n,8] fp32 ([n,16] with num_features = 16)                */
  float *mlp_weights;     /* neural: [816] fp32 (the variant's weight count otherwise), summed
                                     over all visible Gaussians                                */
  float *sv_sites;        /* SV:     [n,7,7] with respect to the raw site parameters            */
} GsGrads;

/* Create / destroy a context on CUDA device `device`.  The context owns 32 bytes of counters
 * (device and pinned host) and 7.5 MB of device memory for the per-CTA partial sums of the decoder
 * gradient.  Not thread safe: use one context per host thread, and one per stream whose calls may
 * overlap on the GPU.  Returns GS_ERR_CUDA if the device cannot be used. */
GsStatus gs_create(int device, GsContext **ctx);
void gs_destroy(GsContext *ctx);
const char *gs_last_error(const GsContext *ctx);

/* Bytes of scratch the render calls need for n Gaussians, a width x height image and at most
 * pair_capacity (Gaussian, tile) instances.  0 on invalid arguments. */
size_t gs_workspace_bytes(int64_t n, int32_t width, int32_t height, int64_t pair_capacity);

/* Preprocess (Sec. 3.1; fused appearance: Sec. 4 "CUDA Implementation").  For every Gaussian:
 * cull, project (EWA), bound the alpha >= 1/255 ellipse by a tile rectangle and count the tiles
 * inside it that the ellipse reaches, and decode the view-dependent colour for the direction
 * camera centre -> mean (SH: Eq. 1-2; neural: Eq. 5-7; Spherical Voronoi: Eq. 3).  Writes all of `out` and the total instance count to *num_pairs_host (host
 * pointer; the call synchronises the stream once to read it).  n = 0 is valid. */
GsStatus gs_preprocess(GsContext *ctx, const GsScene *scene, const GsCamera *cam, GsProjected *out,
                       int64_t *num_pairs_host, void *stream);

/* The same without the host read: nothing is copied back and the call does not wait for the GPU.
 * The instance count stays in the context, on the device, for the gs_render_forward that follows on
 * the same stream with num_pairs = GS_PAIRS_ON_DEVICE.  With it a whole view (and the next ones, on
 * other streams with contexts of their own) can be queued without the host ever waiting, which is
 * what lets independent views overlap on the GPU.  Not in the paper, whose rasterizer reads the
 * count back as usual. */
GsStatus gs_preprocess_async(GsContext *ctx, const GsScene *scene, const GsCamera *cam, GsProjected *out,
                             void *stream);
/* gs_render_forward / gs_render_backward accept this as num_pairs: the count is the one the
 * context's last gs_preprocess(_async) left on the device.  Buffers and kernel grids are then sized
 * by pair_capacity.  If the true count exceeds pair_capacity the instance lists are cut off at
 * pair_capacity (no write ever leaves the caller's buffers), the image of that view is wrong, and a
 * flag is set that gs_async_status reports. */
#define GS_PAIRS_ON_DEVICE ((int64_t)-1)
/* Waits for `stream`, then returns GS_ERR_CAPACITY if any device-counted view on this context
 * overflowed its pair_capacity since the last call (and clears the flag), GS_ERR_INTERNAL if a kernel
 * gave up a bounded wait on one of its own bulk copies (never expected; the waits exist so that a
 * kernel cannot hang), else GS_OK. */
GsStatus gs_async_status(GsContext *ctx, void *stream);

/* Tile assignment, ordering and blending (Sec. 3.1, blend kernel).  Orders the visible
 * Gaussians by depth, emits one instance per (Gaussian, tile), orders instances by tile keeping
 * the depth order, records per-tile ranges, then composites every pixel front to back:
 * alpha = min(0.99, o exp(-0.5 d^T Q d)), skipped below 1/255, stop before transmittance would
 * fall below 1e-4.  image [3,H,W], final_T [H,W] (transmittance left), n_contrib [H,W] (1 + list
 * position of the last composited instance).  GS_ERR_CAPACITY, with nothing written, if
 * num_pairs > pair_capacity or the workspace is smaller than gs_workspace_bytes(). */
GsStatus gs_render_forward(GsContext *ctx, int64_t n, const GsProjected *proj, const GsCamera *cam,
                           int64_t num_pairs, int64_t pair_capacity, GsBinning *bin, float *image,
                           float *final_T, uint32_t *n_contrib, void *workspace,
                           size_t workspace_bytes, void *stream);

/* Backward of the blend and of the preprocess, appearance included (Sec. 4 "CUDA
 * Implementation": the directional colour gradient also reaches the means).  `final_T` and
 * `n_contrib` are the forward's outputs for the same view, dL_dimage is [3,H,W].  Fills every
 * member of `grads` that applies to scene->app.  Uses the same workspace (contents of the forward
 * call are not needed). */
GsStatus gs_render_backward(GsContext *ctx, const GsScene *scene, const GsCamera *cam,
                            const GsProjected *proj, const GsBinning *bin, int64_t num_pairs,
                            const float *final_T, const uint32_t *n_contrib, const float *dL_dimage,
                            GsGrads *grads, void *workspace, size_t workspace_bytes, void *stream);

/* The separate-pass appearance path (Sec. 4 "CUDA Implementation", reference path; App. B.2):
 * colour decode for given unit directions dirs [n,3] without the rasterizer, and its backward.
 * Only the appearance members of `scene` are read.  color [n,3].  gs_appearance_backward fills
 * grads->base_color, grads->sh_rest or grads->features + grads->mlp_weights or grads->sv_sites, and dL_ddirs
 * [n,3] (gradient with respect to the direction as a free vector). */
GsStatus gs_appearance_forward(GsContext *ctx, const GsScene *scene, const float *dirs, float *color,
                               void *stream);
GsStatus gs_appearance_backward(GsContext *ctx, const GsScene *scene, const float *dirs,
                                const float *dL_dcolor, GsGrads *grads, float *dL_ddirs,
                                void *stream);

/* gs_appearance_backward for callers that cannot allocate device memory (the paper has no
 * counterpart; this entry point exists for integration only).  It is meant for code that runs where
 * cudaMalloc is not an option: a plugin inside a host application that owns the whole memory budget
 * and forbids allocations after start-up, a latency-critical loop that may not take the allocator's
 * implicit synchronisation, or a process that cannot afford gs_create (which allocates the context's
 * buffers).  It needs no GsContext, and it calls no cudaMalloc, cudaFree or any allocating library
 * routine.  Neural appearance only (the SH backward uses no scratch: call gs_appearance_backward).
 *
 * The scratch the kernel needs - one row of 816 fp32 partial sums of the decoder-weight gradient per
 * CTA - is a static device array compiled into the library: 1024 rows = 3,342,336 bytes, held by
 * every GPU that loads the library until the process exits.  A launch has at most 1024 CTAs, each
 * covering at most 32 x 128 Gaussians, so n may be at most 4,194,304; a larger n is rejected with
 * GS_ERR_CAPACITY and a message, nothing launched.  Arguments and results are those of
 * gs_appearance_backward (device pointers on the CURRENT device, 16-byte aligned), including
 * scene->color_activation and scene->decoder_precision (GS_DECODER_HALF runs the same unsplit kernel
 * as there; an unknown value of either is GS_ERR_INVALID_ARG); it always runs the warp-level MMA
 * kernel: per-Gaussian results are bit-identical to gs_appearance_backward under
 * GS_ENGINE_WARP_MMA, grads->mlp_weights is the same sum taken in a different order.  error_text
 * (host, may be NULL) receives a description when the status is not GS_OK.
 *
 * The first call on each device looks up the device address of the array; make that call before any
 * stream capture begins.  All calls share the one array, which keeps the previous call's values:
 * every row a launch reads is first overwritten in full by that launch, so nothing needs clearing,
 * but two calls that overlap on the GPU (different streams, or one device used from two threads)
 * race on it and give wrong weight gradients - serialise them. */
GsStatus gs_appearance_backward_noalloc(const GsScene *scene, const float *dirs, const float *dL_dcolor,
                                        GsGrads *grads, float *dL_ddirs, void *stream, char *error_text,
                                        size_t error_text_bytes);

/* ---- NEXT step after the rendering path: the fused Adam update (App. C.1, App. C.2) ------------
 * The paper's optimiser is Adam with one change: it takes ONE LEARNING RATE PER COLUMN of a
 * parameter tensor (App. C.1), so that e.g. base colour, coefficients or the parameters of a site
 * keep their own rates without being split into separate tensors.  Features and decoder weights are
 * stored and updated in single precision, and a half-precision copy is made for the next
 * iteration's forward and backward pass (App. C.2).  The update touches every row, also those of
 * Gaussians that were invisible this iteration (Tab. 3, footnote).
 *
 * One tensor of an update, row-major [rows, cols]:
 *   m <- beta1 m + (1 - beta1) g;   v <- beta2 v + (1 - beta2) g^2;
 *   param <- param - lr[c] (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps)
 * param, grad, exp_avg (m), exp_avg_sq (v): DEVICE pointers, fp32, 16-byte aligned, owned by the
 * caller; param, exp_avg, exp_avg_sq are updated in place, grad is only read.  half_copy: DEVICE
 * pointer to [rows, cols] IEEE fp16 bits (8-byte aligned) that receives the updated values rounded
 * to nearest even, or NULL.  lr: HOST array of cols rates (read during the call).  A decoder-weight
 * vector is a tensor with rows = 816, cols = 1 (App. B.2 sets its beta2 to 0.99). */
enum { GS_ADAM_MAX_COLS = 64, GS_ADAM_MAX_TENSORS = 8, GS_ADAM_MAX_MORE_GRADS = 7 };
typedef struct {
  float *param;
  const float *grad;
  float *exp_avg;
  float *exp_avg_sq;
  uint16_t *half_copy;
  int64_t rows;
  int32_t cols;          /* 1 .. GS_ADAM_MAX_COLS; rows * cols < 2^32 */
  const float *lr;
  float beta1, beta2, eps;
  const float *const *more_grads; /* HOST array of num_more_grads DEVICE pointers, each [rows, cols] fp32 and
                                     16-byte aligned, or NULL: the gradient of the step is grad plus these
                                     (the views of an iteration, each with a gradient buffer of its own)  */
  int32_t num_more_grads;         /* 0 .. GS_ADAM_MAX_MORE_GRADS                                           */
} GsAdamTensor;
/* Updates up to GS_ADAM_MAX_TENSORS tensors with ONE kernel launch on `stream` (asynchronous; no
 * allocation, no synchronisation).  step = 1, 2, ... is the number of this update, shared by the
 * tensors.  Tensors with rows = 0 are skipped.  GS_ERR_INVALID_ARG (nothing launched) for a NULL or
 * misaligned pointer, cols out of range, step < 1, betas outside [0, 1) or too many tensors;
 * GS_ERR_CAPACITY if a tensor has 2^32 elements or more. */
GsStatus gs_adam_step(GsContext *ctx, const GsAdamTensor *tensors, int32_t num_tensors, int64_t step, void *stream);

/* ---- NEXT: the viewer's colour prepass of the neural model as CUDA kernels (App. C.3, "Neural") --
 * Export: gs_neural_fold folds the 17 view-independent columns of the decoder's first layer (the 16
 * encoded feature inputs and the constant degree-0 input) into 16 half-precision pre-activations per
 * Gaussian, stored in place of the features' encodings (32 B per Gaussian).  scene->features,
 * scene->mlp_weights and preact [n,16] (IEEE fp16 bits, 16-byte aligned) are device pointers.
 *
 * Per frame: gs_neural_prepass evaluates what depends on the view - the 15 direction columns of the
 * first layer (SH degrees 1..active_degree of d = normalize(mean - camera centre)), the second and
 * the output layer, 560 instead of 816 multiply-accumulates per Gaussian - in half precision with
 * fp32 accumulation, composes the residual with the base colour, c = max(0, c0 + 0.5 + tanh(.)), and
 * writes one texel per Gaussian: rgba [n,4] bytes = (c clamped to [0,1], sigmoid(opacity logit)),
 * each times 255 and rounded to nearest.  color (optional, may be NULL) receives the unquantised
 * colour [n,3] fp32.  Uses scene->n, means, opacity_logits, base_color, mlp_weights, active_degree
 * (0 disables the residual); of the camera only its centre matters.  Asynchronous on `stream`;
 * GS_ERR_INVALID_ARG for NULL or misaligned pointers, GS_ERR_UNSUPPORTED for a scene that is not
 * GS_APP_NEURAL.  The WebGL viewer itself is out of reach here; this is its shader arithmetic. */
GsStatus gs_neural_fold(GsContext *ctx, const GsScene *scene, uint16_t *preact, void *stream);
GsStatus gs_neural_prepass(GsContext *ctx, const GsScene *scene, const uint16_t *preact, const GsCamera *cam,
                           uint8_t *rgba, float *color, void *stream);

/* Per-stage device timing, for benchmarks (the paper gives wall-clock protocols only, App. C; this
 * is the measurement hook of this library).  While enabled, every stage the library launches is
 * bracketed by CUDA events on the caller's stream and by an NVTX range named after the stage (for a tracing
 * tool; a no-op without one).  gs_profile_collect synchronises those events,
 * ADDS the elapsed milliseconds and the kernel-launch counts since the last collect into
 * ms[GS_NUM_STAGES] / launches[GS_NUM_STAGES] (host arrays, either may be NULL) and forgets them.
 * At most 4096 stage records are kept between two collects; further ones are dropped. */
typedef enum {
  GS_STAGE_PREPROCESS_FWD = 0, /* projection + fused colour decode                              */
  GS_STAGE_DEPTH_SORT,         /* radix sort of the Gaussians by depth key                      */
  GS_STAGE_TILE_OFFSETS,       /* (the sums of tiles touched are taken by the depth sort's last pass: no time of its own) */
  GS_STAGE_KEYGEN,             /* instance emission                                             */
  GS_STAGE_TILE_SORT,          /* radix sort of the instances by tile id                        */
  GS_STAGE_TILE_RANGES,
  GS_STAGE_BLEND_FWD,
  GS_STAGE_BLEND_BWD,
  GS_STAGE_PREPROCESS_BWD,     /* projection backward + fused appearance backward               */
  GS_STAGE_APPEARANCE_FWD,     /* separate-pass decode                                          */
  GS_STAGE_APPEARANCE_BWD,
  GS_STAGE_ADAM,               /* fused parameter update                                        */
  GS_STAGE_PREPASS,            /* viewer-side fold / colour prepass                             */
  GS_NUM_STAGES
} GsStage;
GsStatus gs_profile_enable(GsContext *ctx, int enable);
/* Which kernels evaluate the default decoder (Eq. 5-7) in the separate pass of this context
 * (gs_appearance_forward / gs_appearance_backward, and the appearance passes of gs_preprocess and
 * gs_render_backward when GsScene.separate_pass is set).
 * GS_ENGINE_WARP_MMA: warp-level mma.sync tiles, 32 Gaussians per warp.
 * GS_ENGINE_TCGEN05: tcgen05.mma with the accumulators in tensor memory, 128 Gaussians per CTA, one
 * operand row and one lane of tensor memory per thread; in the backward the weight gradients are
 * products over the 128 Gaussians of a tile, accumulated in tensor memory across the CTA's tiles.
 * GS_ENGINE_AUTO (the default): per kernel, whichever measured faster on a B200 - the backward with
 * split operands and, from 2,000,000 Gaussians on, the forward on tcgen05; smaller forwards and the
 * plain-fp16 backward on warp-level MMA.
 * Same arithmetic (fp16 operands, split or plain, fp32 accumulation) and the same tolerances either
 * way; per-Gaussian results differ only by the order of the fp32 sums.
 * A decoder of another size (GsScene.mlp_hidden / mlp_layers / num_features, App. D's architecture
 * table) runs on tcgen05 kernels of the same construction under GS_ENGINE_TCGEN05 and GS_ENGINE_AUTO -
 * inside gs_render_backward they work on the Gaussians that received a gradient only - and on fp32
 * FMA kernels (dense over all Gaussians) under GS_ENGINE_WARP_MMA; same tolerances.  The paper has
 * no counterpart of this call.  Returns GS_ERR_INVALID_ARG for any other value.  Takes effect for the calls issued
 * after it. */
typedef enum GsDecoderEngine { GS_ENGINE_WARP_MMA = 0, GS_ENGINE_TCGEN05 = 1, GS_ENGINE_AUTO = 2 } GsDecoderEngine;
GsStatus gs_set_decoder_engine(GsContext *ctx, int engine);
/* Measurement only: for the view last rendered into (proj, bin), count over all pixels the list
 * entries the blend evaluates (until each pixel stops) and the pairs it composites; these are the
 * work units of the blend kernels' roofline.  counts_host is a host array of FOUR values: entries
 * evaluated, pairs composited, (warp, entry) steps the forward walks (a warp covers 16 x 8 pixels)
 * and the steps among them in which no pixel of the warp accepts the entry.  Synchronises. */
GsStatus gs_profile_blend_counts(GsContext *ctx, const GsProjected *proj, const GsBinning *bin, const GsCamera *cam,
                                 int64_t *counts_host, void *stream);
GsStatus gs_profile_collect(GsContext *ctx, double *ms, int64_t *launches);

#ifdef __cplusplus
}
#endif
#endif /* GS_B200_H_ */
