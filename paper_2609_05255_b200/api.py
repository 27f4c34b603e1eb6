"""Thin ctypes binding of ``libgs_b200.so`` (the C ABI declared in ``include/gs.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.
PyTorch supplies device memory and streams.  There is no CPU fallback: importing this module
fails loudly if the shared library has not been built (``python -m paper_2609_05255_b200.build``).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgs_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_05255_b200.build` "
                      "(there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

GS_OK, GS_ERR_INVALID_ARG, GS_ERR_CAPACITY, GS_ERR_CUDA, GS_ERR_UNSUPPORTED, GS_ERR_INTERNAL = 0, -1, -2, -3, -4, -6
GS_APP_SH, GS_APP_NEURAL, GS_APP_SV = 0, 1, 2
GS_DECODER_SPLIT, GS_DECODER_HALF = 0, 1
TILE = 16
MLP_WEIGHTS = 816

_vp = C.c_void_p


class GsCamera(C.Structure):
    _fields_ = [("width", C.c_int32), ("height", C.c_int32), ("fx", C.c_float), ("fy", C.c_float),
                ("cx", C.c_float), ("cy", C.c_float), ("w2c", C.c_float * 12), ("near_plane", C.c_float),
                ("far_plane", C.c_float), ("background", C.c_float * 3)]


class GsScene(C.Structure):
    _fields_ = [("n", C.c_int64), ("means", _vp), ("log_scales", _vp), ("quats", _vp), ("opacity_logits", _vp),
                ("base_color", _vp), ("app", C.c_int32), ("active_degree", C.c_int32), ("sh_rest", _vp),
                ("features", _vp), ("mlp_weights", _vp), ("color_activation", C.c_int32), ("sv_sites", _vp),
                ("mlp_hidden", C.c_int32), ("mlp_layers", C.c_int32), ("num_features", C.c_int32),
                ("separate_pass", C.c_int32), ("decoder_precision", C.c_int32)]


class GsProjected(C.Structure):
    _fields_ = [("mean2d", _vp), ("conic_opacity", _vp), ("color", _vp), ("depth_key", _vp), ("rect", _vp),
                ("tiles_touched", _vp), ("extent", _vp), ("cell_count", _vp), ("cell_records", _vp)]


class GsBinning(C.Structure):
    _fields_ = [("depth_order", _vp), ("sorted_tiles", _vp), ("sorted_vals", _vp), ("tile_ranges", _vp),
                ("tile_order", _vp)]


class GsGrads(C.Structure):
    _fields_ = [("means", _vp), ("log_scales", _vp), ("quats", _vp), ("opacity_logits", _vp), ("base_color", _vp),
                ("sh_rest", _vp), ("features", _vp), ("mlp_weights", _vp), ("sv_sites", _vp)]


_lib.gs_create.argtypes = [C.c_int, C.POINTER(_vp)]
_lib.gs_create.restype = C.c_int
_lib.gs_destroy.argtypes = [_vp]
_lib.gs_destroy.restype = None
_lib.gs_last_error.argtypes = [_vp]
_lib.gs_last_error.restype = C.c_char_p
_lib.gs_workspace_bytes.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int64]
_lib.gs_workspace_bytes.restype = C.c_size_t
_lib.gs_preprocess.argtypes = [_vp, C.POINTER(GsScene), C.POINTER(GsCamera), C.POINTER(GsProjected),
                               C.POINTER(C.c_int64), _vp]
_lib.gs_preprocess.restype = C.c_int
_lib.gs_preprocess_async.argtypes = [_vp, C.POINTER(GsScene), C.POINTER(GsCamera), C.POINTER(GsProjected), _vp]
_lib.gs_preprocess_async.restype = C.c_int
_lib.gs_async_status.argtypes = [_vp, _vp]
_lib.gs_async_status.restype = C.c_int
GS_PAIRS_ON_DEVICE = -1
_lib.gs_render_forward.argtypes = [_vp, C.c_int64, C.POINTER(GsProjected), C.POINTER(GsCamera), C.c_int64,
                                   C.c_int64, C.POINTER(GsBinning), _vp, _vp, _vp, _vp, C.c_size_t, _vp]
_lib.gs_render_forward.restype = C.c_int
_lib.gs_render_backward.argtypes = [_vp, C.POINTER(GsScene), C.POINTER(GsCamera), C.POINTER(GsProjected),
                                    C.POINTER(GsBinning), C.c_int64, _vp, _vp, _vp, C.POINTER(GsGrads), _vp,
                                    C.c_size_t, _vp]
_lib.gs_render_backward.restype = C.c_int
_lib.gs_appearance_forward.argtypes = [_vp, C.POINTER(GsScene), _vp, _vp, _vp]
_lib.gs_appearance_forward.restype = C.c_int
_lib.gs_appearance_backward.argtypes = [_vp, C.POINTER(GsScene), _vp, _vp, C.POINTER(GsGrads), _vp, _vp]
_lib.gs_appearance_backward.restype = C.c_int


STAGES = ["preprocess_fwd", "depth_sort", "tile_offsets", "keygen", "tile_sort", "tile_ranges", "blend_fwd",
          "blend_bwd", "preprocess_bwd", "appearance_fwd", "appearance_bwd", "adam", "prepass"]
_lib.gs_profile_enable.argtypes = [_vp, C.c_int]
_lib.gs_profile_enable.restype = C.c_int
_lib.gs_profile_collect.argtypes = [_vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
_lib.gs_profile_collect.restype = C.c_int


_lib.gs_set_decoder_engine.argtypes = [_vp, C.c_int]
_lib.gs_set_decoder_engine.restype = C.c_int
_lib.gs_profile_blend_counts.argtypes = [_vp, C.POINTER(GsProjected), C.POINTER(GsBinning), C.POINTER(GsCamera),
                                         C.POINTER(C.c_int64), _vp]
_lib.gs_profile_blend_counts.restype = C.c_int


GS_ADAM_MAX_COLS, GS_ADAM_MAX_TENSORS = 64, 8


class GsAdamTensor(C.Structure):
    _fields_ = [("param", _vp), ("grad", _vp), ("exp_avg", _vp), ("exp_avg_sq", _vp), ("half_copy", _vp),
                ("rows", C.c_int64), ("cols", C.c_int32), ("lr", C.POINTER(C.c_float)), ("beta1", C.c_float),
                ("beta2", C.c_float), ("eps", C.c_float), ("more_grads", C.POINTER(_vp)), ("num_more_grads", C.c_int32)]


_lib.gs_adam_step.argtypes = [_vp, C.POINTER(GsAdamTensor), C.c_int32, C.c_int64, _vp]
_lib.gs_adam_step.restype = C.c_int
_lib.gs_neural_fold.argtypes = [_vp, C.POINTER(GsScene), _vp, _vp]
_lib.gs_neural_fold.restype = C.c_int
_lib.gs_neural_prepass.argtypes = [_vp, C.POINTER(GsScene), _vp, C.POINTER(GsCamera), _vp, _vp, _vp]
_lib.gs_neural_prepass.restype = C.c_int


class GsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gs status {status}: {message}")
        self.status = status


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device pointers must come from contiguous CUDA tensors"
    return t.data_ptr()


def _stream_handle(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def make_camera(cam) -> GsCamera:
    """Any object with width, height, fx, fy, cx, cy, w2c[3,4], near_plane, far_plane, background."""
    c = GsCamera()
    c.width, c.height = int(cam.width), int(cam.height)
    c.fx, c.fy, c.cx, c.cy = float(cam.fx), float(cam.fy), float(cam.cx), float(cam.cy)
    c.w2c = (C.c_float * 12)(*np.asarray(cam.w2c, np.float32).reshape(12).tolist())
    c.near_plane, c.far_plane = float(cam.near_plane), float(cam.far_plane)
    c.background = (C.c_float * 3)(*[float(v) for v in cam.background])
    return c


@dataclass
class DeviceScene:
    """The scene's tensors on the device (fp32; features / weights fp16)."""
    means: torch.Tensor
    log_scales: torch.Tensor
    quats: torch.Tensor
    opacity_logits: torch.Tensor
    base_color: torch.Tensor
    app: int
    active_degree: int
    sh_rest: Optional[torch.Tensor] = None
    features: Optional[torch.Tensor] = None
    mlp_weights: Optional[torch.Tensor] = None
    color_activation: int = 0        # GS_ACT_*: 0 ReLU(x+0.5), 1 softplus beta 10, 2 sigmoid(4x), 3 clamp(x+0.5, 0, 1)
    sv_sites: Optional[torch.Tensor] = None      # Spherical Voronoi: [n,7,7]
    mlp_hidden: int = 16             # decoder architecture (App. D); anything but 16 / 2 / 8 runs in
    mlp_layers: int = 2              # gs_appearance_forward / backward only
    num_features: int = 8
    separate_pass: int = 0           # 1: the unfused reference path (appearance as passes of its own)
    decoder_precision: int = 0       # 0: split fp16 operands (fp32-accurate); 1: plain fp16 operands (the paper's)

    @property
    def n(self) -> int:
        return int(self.base_color.shape[0])

    def c_struct(self) -> GsScene:
        s = GsScene()
        s.n = self.n
        s.means, s.log_scales, s.quats = _ptr(self.means), _ptr(self.log_scales), _ptr(self.quats)
        s.opacity_logits, s.base_color = _ptr(self.opacity_logits), _ptr(self.base_color)
        s.app, s.active_degree = int(self.app), int(self.active_degree)
        s.sh_rest, s.features, s.mlp_weights = _ptr(self.sh_rest), _ptr(self.features), _ptr(self.mlp_weights)
        s.color_activation = int(self.color_activation)
        s.sv_sites = _ptr(self.sv_sites)
        s.mlp_hidden, s.mlp_layers, s.num_features = int(self.mlp_hidden), int(self.mlp_layers), int(self.num_features)
        s.separate_pass = int(self.separate_pass)
        s.decoder_precision = int(self.decoder_precision)
        return s


def upload_scene(scene, device="cuda") -> DeviceScene:
    """Copy a host scene (numpy arrays, see scenes.Scene) to the device."""
    def up(a, dtype):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=dtype)
    return DeviceScene(up(scene.means, torch.float32), up(scene.log_scales, torch.float32),
                       up(scene.quats, torch.float32), up(scene.opacity_logits, torch.float32),
                       up(scene.base_color, torch.float32), int(scene.app), int(scene.active_degree),
                       up(scene.sh_rest, torch.float32), up(scene.features, torch.float16),
                       up(scene.mlp_weights, torch.float16), int(getattr(scene, "color_activation", 0)),
                       up(getattr(scene, "sv_sites", None), torch.float32),
                       int(getattr(scene, "mlp_hidden", 0)) or 16, int(getattr(scene, "mlp_layers", 0)) or 2,
                       int(scene.features.shape[1]) if scene.features is not None else 8,
                       int(getattr(scene, "separate_pass", 0)), int(getattr(scene, "decoder_precision", 0)))


@dataclass
class Projected:
    mean2d: torch.Tensor
    conic_opacity: torch.Tensor
    color: torch.Tensor
    depth_key: torch.Tensor    # int32 storage holding the uint32 bit patterns
    rect: torch.Tensor         # int16 storage holding uint16 tile coordinates, [n,4]
    tiles_touched: torch.Tensor
    extent: Optional[torch.Tensor]
    cell_count: torch.Tensor = None      # [n]   footprint by cells of 4 x 4 tiles: opaque, for gs_render_forward
    cell_records: torch.Tensor = None    # [n,9]

    def c_struct(self) -> GsProjected:
        p = GsProjected()
        p.mean2d, p.conic_opacity, p.color = _ptr(self.mean2d), _ptr(self.conic_opacity), _ptr(self.color)
        p.depth_key, p.rect, p.extent = _ptr(self.depth_key), _ptr(self.rect), _ptr(self.extent)
        p.tiles_touched = _ptr(self.tiles_touched)
        p.cell_count, p.cell_records = _ptr(self.cell_count), _ptr(self.cell_records)
        return p


def alloc_projected(n: int, device, with_extent: bool = True) -> Projected:
    m = max(n, 1)
    f = dict(device=device, dtype=torch.float32)
    return Projected(torch.empty((m, 2), **f), torch.empty((m, 4), **f), torch.empty((m, 3), **f),
                     torch.empty((m,), device=device, dtype=torch.int32),
                     torch.empty((m, 4), device=device, dtype=torch.int16),
                     torch.empty((m,), device=device, dtype=torch.int32),
                     torch.empty((m, 4), **f) if with_extent else None,
                     torch.empty((m,), device=device, dtype=torch.int32),
                     torch.empty((m, 9), device=device, dtype=torch.int32))


@dataclass
class Binning:
    depth_order: torch.Tensor
    sorted_tiles: torch.Tensor
    sorted_vals: torch.Tensor
    tile_ranges: torch.Tensor
    tile_order: torch.Tensor

    def c_struct(self) -> GsBinning:
        b = GsBinning()
        b.depth_order, b.sorted_tiles = _ptr(self.depth_order), _ptr(self.sorted_tiles)
        b.sorted_vals, b.tile_ranges = _ptr(self.sorted_vals), _ptr(self.tile_ranges)
        b.tile_order = _ptr(self.tile_order)
        return b


def alloc_binning(n: int, pair_capacity: int, width: int, height: int, device) -> Binning:
    tiles = ((width + TILE - 1) // TILE) * ((height + TILE - 1) // TILE)
    i = dict(device=device, dtype=torch.int32)
    return Binning(torch.empty((max(n, 1),), **i), torch.empty((max(pair_capacity, 1),), **i),
                   torch.empty((max(pair_capacity, 1),), **i), torch.empty((tiles, 2), **i),
                   torch.empty((tiles,), **i))


@dataclass
class Grads:
    means: torch.Tensor
    log_scales: torch.Tensor
    quats: torch.Tensor
    opacity_logits: torch.Tensor
    base_color: torch.Tensor
    sh_rest: Optional[torch.Tensor] = None
    features: Optional[torch.Tensor] = None
    mlp_weights: Optional[torch.Tensor] = None
    sv_sites: Optional[torch.Tensor] = None

    def c_struct(self) -> GsGrads:
        g = GsGrads()
        g.means, g.log_scales, g.quats = _ptr(self.means), _ptr(self.log_scales), _ptr(self.quats)
        g.opacity_logits, g.base_color = _ptr(self.opacity_logits), _ptr(self.base_color)
        g.sh_rest, g.features, g.mlp_weights = _ptr(self.sh_rest), _ptr(self.features), _ptr(self.mlp_weights)
        g.sv_sites = _ptr(self.sv_sites)
        return g


def decoder_num_weights(hidden: int = 16, layers: int = 2) -> int:
    return 32 * hidden + (layers - 1) * hidden * hidden + 3 * hidden


def alloc_grads(n: int, app: int, device, num_features: int = 8, num_weights: int = MLP_WEIGHTS) -> Grads:
    m = max(n, 1)
    f = dict(device=device, dtype=torch.float32)
    g = Grads(torch.empty((m, 3), **f), torch.empty((m, 3), **f), torch.empty((m, 4), **f),
              torch.empty((m,), **f), torch.empty((m, 3), **f))
    if app == GS_APP_SH:
        g.sh_rest = torch.empty((m, 15, 3), **f)
    elif app == GS_APP_SV:
        g.sv_sites = torch.empty((m, 7, 7), **f)
    else:
        g.features = torch.empty((m, num_features), **f)
        g.mlp_weights = torch.empty((num_weights,), **f)
    return g


def alloc_grads_for(scene: DeviceScene, device) -> Grads:
    """Gradient buffers shaped for the scene's appearance model and decoder."""
    return alloc_grads(scene.n, scene.app, device, scene.num_features,
                       decoder_num_weights(scene.mlp_hidden, scene.mlp_layers))


class Context:
    """Owner of one GsContext (gs_create / gs_destroy)."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self.device = torch.device("cuda", device)
        h = _vp()
        st = _lib.gs_create(device, C.byref(h))
        if st != GS_OK:
            raise GsError(st, "gs_create failed")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            _lib.gs_destroy(self._h)
            self._h = None

    __del__ = close

    def _check(self, st: int):
        if st != GS_OK:
            raise GsError(st, _lib.gs_last_error(self._h).decode())


def gs_profile_enable(ctx: Context, enable: bool) -> None:
    ctx._check(_lib.gs_profile_enable(ctx._h, int(enable)))


def gs_profile_collect(ctx: Context):
    """Returns ({stage: milliseconds}, {stage: kernel launches}) accumulated since the last collect."""
    ms = (C.c_double * len(STAGES))()
    launches = (C.c_int64 * len(STAGES))()
    ctx._check(_lib.gs_profile_collect(ctx._h, ms, launches))
    return dict(zip(STAGES, list(ms))), dict(zip(STAGES, list(launches)))


GS_ENGINE_WARP_MMA, GS_ENGINE_TCGEN05, GS_ENGINE_AUTO = 0, 1, 2


def gs_set_decoder_engine(ctx: Context, engine: int):
    ctx._check(_lib.gs_set_decoder_engine(ctx._h, int(engine)))


def gs_profile_blend_counts(ctx: Context, proj: "Projected", binning: "Binning", cam: GsCamera, stream=None):
    """(list entries evaluated, pairs composited, warp steps, warp steps without a taker) over all pixels of the view
    held in proj / binning."""
    out = (C.c_int64 * 4)()
    pp, bb = proj.c_struct(), binning.c_struct()
    ctx._check(_lib.gs_profile_blend_counts(ctx._h, C.byref(pp), C.byref(bb), C.byref(cam), out,
                                            _stream_handle(stream)))
    return int(out[0]), int(out[1]), int(out[2]), int(out[3])


def gs_workspace_bytes(n: int, width: int, height: int, pair_capacity: int) -> int:
    return int(_lib.gs_workspace_bytes(n, width, height, pair_capacity))


def gs_preprocess(ctx: Context, scene: DeviceScene, cam: GsCamera, out: Projected, stream=None) -> int:
    """Returns the number of (Gaussian, tile) instances; synchronises the stream once."""
    pairs = C.c_int64(0)
    cs, po = scene.c_struct(), out.c_struct()
    ctx._check(_lib.gs_preprocess(ctx._h, C.byref(cs), C.byref(cam), C.byref(po), C.byref(pairs),
                                  _stream_handle(stream)))
    return int(pairs.value)


def gs_preprocess_async(ctx: Context, scene: "DeviceScene", cam: GsCamera, out: "Projected", stream=None) -> None:
    """gs_preprocess without the host read of the instance count (it stays on the device, see GS_PAIRS_ON_DEVICE)."""
    cs, pp = scene.c_struct(), out.c_struct()
    ctx._check(_lib.gs_preprocess_async(ctx._h, C.byref(cs), C.byref(cam), C.byref(pp), _stream_handle(stream)))


def gs_async_status(ctx: Context, stream=None) -> None:
    """Wait for the stream; raise GsError(GS_ERR_CAPACITY) if a device-counted view overflowed its capacity."""
    ctx._check(_lib.gs_async_status(ctx._h, _stream_handle(stream)))


def gs_render_forward(ctx: Context, n: int, proj: Projected, cam: GsCamera, num_pairs: int, pair_capacity: int,
                      binning: Binning, image: torch.Tensor, final_T: torch.Tensor, n_contrib: torch.Tensor,
                      workspace: torch.Tensor, stream=None) -> None:
    pp, bb = proj.c_struct(), binning.c_struct()
    ctx._check(_lib.gs_render_forward(ctx._h, n, C.byref(pp), C.byref(cam), num_pairs, pair_capacity, C.byref(bb),
                                      _ptr(image), _ptr(final_T), _ptr(n_contrib), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream_handle(stream)))


def gs_render_backward(ctx: Context, scene: DeviceScene, cam: GsCamera, proj: Projected, binning: Binning,
                       num_pairs: int, final_T: torch.Tensor, n_contrib: torch.Tensor, dL_dimage: torch.Tensor,
                       grads: Grads, workspace: torch.Tensor, stream=None) -> None:
    cs, pp, bb, gg = scene.c_struct(), proj.c_struct(), binning.c_struct(), grads.c_struct()
    ctx._check(_lib.gs_render_backward(ctx._h, C.byref(cs), C.byref(cam), C.byref(pp), C.byref(bb), num_pairs,
                                       _ptr(final_T), _ptr(n_contrib), _ptr(dL_dimage), C.byref(gg),
                                       _ptr(workspace), workspace.numel() * workspace.element_size(),
                                       _stream_handle(stream)))


def gs_appearance_forward(ctx: Context, scene: DeviceScene, dirs: torch.Tensor, color: torch.Tensor,
                          stream=None) -> None:
    cs = scene.c_struct()
    ctx._check(_lib.gs_appearance_forward(ctx._h, C.byref(cs), _ptr(dirs), _ptr(color), _stream_handle(stream)))


def gs_appearance_backward(ctx: Context, scene: DeviceScene, dirs: torch.Tensor, dL_dcolor: torch.Tensor,
                           grads: Grads, dL_ddirs: torch.Tensor, stream=None) -> None:
    cs, gg = scene.c_struct(), grads.c_struct()
    ctx._check(_lib.gs_appearance_backward(ctx._h, C.byref(cs), _ptr(dirs), _ptr(dL_dcolor), C.byref(gg),
                                           _ptr(dL_ddirs), _stream_handle(stream)))


# ------------------------------------------------------------------------------------------------
# Convenience: one view, forward + backward, buffers allocated with torch.  Still marshalling only.
# ------------------------------------------------------------------------------------------------
class Renderer:
    """Holds the per-view buffers so that repeated steps allocate nothing."""

    def __init__(self, ctx: Context, n: int, width: int, height: int, app: int, pair_capacity: int,
                 with_extent: bool = False):
        dev = ctx.device
        self.ctx, self.n, self.width, self.height, self.app = ctx, n, width, height, app
        self.pair_capacity = pair_capacity
        self.proj = alloc_projected(n, dev, with_extent)
        self.binning = alloc_binning(n, pair_capacity, width, height, dev)
        self.image = torch.empty((3, height, width), device=dev, dtype=torch.float32)
        self.final_T = torch.empty((height, width), device=dev, dtype=torch.float32)
        self.n_contrib = torch.empty((height, width), device=dev, dtype=torch.int32)
        self.grads = alloc_grads(n, app, dev)
        self.workspace = torch.empty((max(gs_workspace_bytes(n, width, height, pair_capacity), 256),),
                                     device=dev, dtype=torch.uint8)
        self.num_pairs = 0

    def forward(self, scene: DeviceScene, cam: GsCamera, stream=None) -> torch.Tensor:
        self.num_pairs = gs_preprocess(self.ctx, scene, cam, self.proj, stream)
        gs_render_forward(self.ctx, scene.n, self.proj, cam, self.num_pairs, self.pair_capacity, self.binning,
                          self.image, self.final_T, self.n_contrib, self.workspace, stream)
        return self.image

    def forward_async(self, scene: DeviceScene, cam: GsCamera, stream=None) -> torch.Tensor:
        """forward() without any host wait: the instance count stays on the device and the lists are sized by
        pair_capacity.  Check gs_async_status(ctx, stream) once the work is done."""
        gs_preprocess_async(self.ctx, scene, cam, self.proj, stream)
        self.num_pairs = GS_PAIRS_ON_DEVICE
        gs_render_forward(self.ctx, scene.n, self.proj, cam, GS_PAIRS_ON_DEVICE, self.pair_capacity, self.binning,
                          self.image, self.final_T, self.n_contrib, self.workspace, stream)
        return self.image

    def backward(self, scene: DeviceScene, cam: GsCamera, dL_dimage: torch.Tensor, stream=None) -> Grads:
        gs_render_backward(self.ctx, scene, cam, self.proj, self.binning, self.num_pairs, self.final_T,
                           self.n_contrib, dL_dimage, self.grads, self.workspace, stream)
        return self.grads


# ------------------------------------------------------------------------------------------------
# Viewer-side colour prepass of the neural model
# ------------------------------------------------------------------------------------------------
def gs_neural_fold(ctx: Context, scene: "DeviceScene", preact: torch.Tensor, stream=None) -> None:
    """preact: [n,16] float16 tensor that receives the folded first-layer pre-activations."""
    cs = scene.c_struct()
    ctx._check(_lib.gs_neural_fold(ctx._h, C.byref(cs), _ptr(preact), _stream_handle(stream)))


def gs_neural_prepass(ctx: Context, scene: "DeviceScene", preact: torch.Tensor, cam: GsCamera, rgba: torch.Tensor,
                      color: Optional[torch.Tensor] = None, stream=None) -> None:
    """rgba: [n,4] uint8 texels; color: optional [n,3] float32 unquantised colour."""
    cs = scene.c_struct()
    ctx._check(_lib.gs_neural_prepass(ctx._h, C.byref(cs), _ptr(preact), C.byref(cam), _ptr(rgba), _ptr(color),
                                      _stream_handle(stream)))


# ------------------------------------------------------------------------------------------------
# Fused Adam update
# ------------------------------------------------------------------------------------------------
class AdamTensor:
    """One parameter tensor of an update: fp32 param / grad / exp_avg / exp_avg_sq of the same shape
    (viewed as [rows, cols] with cols = len(lr)), an optional fp16 tensor that receives the updated
    values, and the hyper-parameters.  Marshalling only."""

    def __init__(self, param, grad, exp_avg, exp_avg_sq, lr, beta1=0.9, beta2=0.999, eps=1e-15, half_copy=None,
                 more_grads=()):
        lr = [float(x) for x in (lr if hasattr(lr, "__len__") else [lr])]
        self.cols = len(lr)
        assert param.numel() % self.cols == 0
        self.rows = param.numel() // self.cols
        self.param, self.grad, self.exp_avg, self.exp_avg_sq, self.half_copy = param, grad, exp_avg, exp_avg_sq, half_copy
        self.lr = (C.c_float * self.cols)(*lr)          # host array, kept alive by this object
        self.beta1, self.beta2, self.eps = beta1, beta2, eps
        self.more_grads = list(more_grads)                       # further gradient tensors, summed with grad
        self._more = (_vp * max(1, len(self.more_grads)))(*[_ptr(g) for g in self.more_grads])

    def c_struct(self) -> GsAdamTensor:
        t = GsAdamTensor()
        t.param, t.grad, t.exp_avg, t.exp_avg_sq = _ptr(self.param), _ptr(self.grad), _ptr(self.exp_avg), _ptr(self.exp_avg_sq)
        t.half_copy = _ptr(self.half_copy)
        t.rows, t.cols, t.lr = self.rows, self.cols, C.cast(self.lr, C.POINTER(C.c_float))
        t.beta1, t.beta2, t.eps = self.beta1, self.beta2, self.eps
        t.more_grads = C.cast(self._more, C.POINTER(_vp)) if self.more_grads else None
        t.num_more_grads = len(self.more_grads)
        return t


def gs_adam_step(ctx: Context, tensors, step: int, stream=None) -> None:
    """Update all `tensors` (AdamTensor objects, at most GS_ADAM_MAX_TENSORS) with one kernel launch."""
    arr = (GsAdamTensor * max(1, len(tensors)))(*[t.c_struct() for t in tensors])
    ctx._check(_lib.gs_adam_step(ctx._h, arr, len(tensors), step, _stream_handle(stream)))


# ------------------------------------------------------------------------------------------------
# The allocation-free neural appearance backward (no context, static device scratch in the library).
# ------------------------------------------------------------------------------------------------
NOALLOC_MAX_N = 4_194_304
_lib.gs_appearance_backward_noalloc.argtypes = [C.POINTER(GsScene), _vp, _vp, C.POINTER(GsGrads), _vp, _vp,
                                                C.c_char_p, C.c_size_t]
_lib.gs_appearance_backward_noalloc.restype = C.c_int


def gs_appearance_backward_noalloc(scene: DeviceScene, dirs: torch.Tensor, dL_dcolor: torch.Tensor,
                                   grads: Grads, dL_ddirs: torch.Tensor, stream=None) -> None:
    """Same results as gs_appearance_backward for the neural model, for callers that may not allocate:
    no Context is needed and the library allocates nothing (its scratch is a static device array, good
    for up to NOALLOC_MAX_N Gaussians).  Calls must not overlap on the GPU; the first call on a device
    should precede any stream capture.  Raises GsError with the library's message on failure."""
    cs, gg = scene.c_struct(), grads.c_struct()
    msg = C.create_string_buffer(256)
    st = _lib.gs_appearance_backward_noalloc(C.byref(cs), _ptr(dirs), _ptr(dL_dcolor), C.byref(gg), _ptr(dL_ddirs),
                                             _stream_handle(stream), msg, len(msg))
    if st != GS_OK:
        raise GsError(st, msg.value.decode())
