"""No kernel writes outside the buffers it is given: every caller-owned buffer of a forward + backward step
(projected arrays, binning arrays with the instance capacity set to exactly the instance count, image-sized
outputs, gradient arrays, the workspace at exactly gs_workspace_bytes) sits between two guard zones filled with
a byte pattern, and the guard zones must come back untouched.  Run for the three appearance models, fused and
through the separate-pass path, and for the device-counted (asynchronous) forward."""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes

pytestmark = pytest.mark.gpu

PAD = 4096          # bytes on either side; a multiple of 256 keeps the payload aligned
PATTERN = 0xA5


class Guarded:
    def __init__(self, torch, device):
        self.torch, self.device, self.blocks = torch, device, []

    def __call__(self, shape, dtype):
        torch = self.torch
        numel = int(np.prod(shape)) if len(shape) else 1
        nbytes = max(numel, 1) * torch.empty((), dtype=dtype).element_size()
        payload = (nbytes + 255) // 256 * 256
        raw = torch.full((PAD + payload + PAD,), PATTERN, dtype=torch.uint8, device=self.device)
        self.blocks.append((raw, payload))
        return raw[PAD:PAD + nbytes].view(dtype).reshape(shape)

    def check(self):
        for k, (raw, payload) in enumerate(self.blocks):
            head, tail = raw[:PAD], raw[PAD + payload:]
            assert bool((head == PATTERN).all()), f"buffer {k}: bytes before it were written"
            assert bool((tail == PATTERN).all()), f"buffer {k}: bytes after it were written"


def step(api, torch, sc, cam, device_count):
    ctx = api.Context(0)
    dev = ctx.device
    ds = api.upload_scene(sc, dev)
    ccam = api.make_camera(cam)
    n, W, H = ds.n, cam.width, cam.height
    tiles = ((W + 15) // 16) * ((H + 15) // 16)
    g = Guarded(torch, dev)
    f32, i32, i16 = torch.float32, torch.int32, torch.int16
    proj = api.Projected(g((n, 2), f32), g((n, 4), f32), g((n, 3), f32), g((n,), i32), g((n, 4), i16), g((n,), i32),
                         g((n, 4), f32), g((n,), i32), g((n, 9), i32))
    P = api.gs_preprocess(ctx, ds, ccam, proj)           # sizes the instance buffers exactly
    assert P > 0
    binning = api.Binning(g((n,), i32), g((P,), i32), g((P,), i32), g((tiles, 2), i32), g((tiles,), i32))
    image, final_T, n_contrib = g((3, H, W), f32), g((H, W), f32), g((H, W), i32)
    ws = g((api.gs_workspace_bytes(n, W, H, P),), torch.uint8)
    grads = api.Grads(g((n, 3), f32), g((n, 3), f32), g((n, 4), f32), g((n,), f32), g((n, 3), f32))
    if ds.app == scenes.APP_SH:
        grads.sh_rest = g((n, 15, 3), f32)
    elif ds.app == scenes.APP_SV:
        grads.sv_sites = g((n, 7, 7), f32)
    else:
        grads.features = g((n, ds.num_features), f32)
        grads.mlp_weights = g((api.decoder_num_weights(ds.mlp_hidden, ds.mlp_layers),), f32)
    G = torch.from_numpy(scenes.upstream_gradient(cam, 5)).to(dev)
    if device_count:
        api.gs_preprocess_async(ctx, ds, ccam, proj)
        api.gs_render_forward(ctx, n, proj, ccam, api.GS_PAIRS_ON_DEVICE, P, binning, image, final_T, n_contrib, ws)
        api.gs_render_backward(ctx, ds, ccam, proj, binning, api.GS_PAIRS_ON_DEVICE, final_T, n_contrib, G, grads, ws)
        api.gs_async_status(ctx)
    else:
        api.gs_render_forward(ctx, n, proj, ccam, P, P, binning, image, final_T, n_contrib, ws)
        api.gs_render_backward(ctx, ds, ccam, proj, binning, P, final_T, n_contrib, G, grads, ws)
    torch.cuda.synchronize()
    g.check()
    assert bool(torch.isfinite(image).all())
    ctx.close()


@pytest.mark.parametrize("app", [scenes.APP_SH, scenes.APP_NEURAL, scenes.APP_SV], ids=["sh", "neural", "sv"])
@pytest.mark.parametrize("mode", ["fused", "separate_pass", "device_count"])
def test_guard_zones_stay_untouched(app, mode):
    import torch
    from paper_2609_05255_b200 import api
    w = scenes.config2(n=10_007, app=app)          # 10 007: a ragged last warp and a ragged last block
    sc = w.scene
    sc.separate_pass = 1 if mode == "separate_pass" else 0
    step(api, torch, sc, w.cameras[0], device_count=(mode == "device_count"))


def test_guard_zones_with_a_decoder_variant_and_a_huge_gaussian():
    import torch
    from paper_2609_05255_b200 import api
    w = scenes.config2(n=4_099, app=scenes.APP_NEURAL)
    sc = w.scene
    rng = np.random.default_rng(np.random.PCG64(6))
    _, sc.features, sc.mlp_weights = scenes.draw_neural_appearance(rng, sc.n, 32, 2, 16)
    sc.mlp_hidden, sc.mlp_layers = 32, 2
    sc.means = sc.means.copy(); sc.log_scales = sc.log_scales.copy()
    sc.means[0] = (0.0, 0.0, 2.5); sc.log_scales[0] = (1.0, 1.0, 1.0)      # covers every tile: the warp-shared emission
    step(api, torch, sc, w.cameras[0], device_count=False)


def test_guard_zones_around_the_adam_update_and_the_viewer_prepass():
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    g = Guarded(torch, dev)
    f32, f16 = torch.float32, torch.float16
    # Adam: odd sizes, a tensor with a half copy and one that sums further gradient sets
    tensors = []
    for rows, cols, half in ((10_007, 3, False), (4_099, 8, True), (816, 1, True), (33, 45, False)):
        p, gr, m, v = (g((rows, cols), f32) for _ in range(4))
        for t, val in ((p, 0.5), (gr, 1e-3), (m, 0.0), (v, 0.0)):
            t.fill_(val)
        more = [g((rows, cols), f32).fill_(2e-3) for _ in range(2)] if cols == 3 else []
        tensors.append(api.AdamTensor(p, gr, m, v, [1e-3] * cols, half_copy=g((rows, cols), f16) if half else None,
                                      more_grads=more))
    api.gs_adam_step(ctx, tensors, 1)
    # viewer prepass: fold + per-frame pass
    w = scenes.config2(n=5_003, app=scenes.APP_NEURAL)
    ds = api.upload_scene(w.scene, dev)
    preact = g((ds.n, 16), f16)
    rgba, color = g((ds.n, 4), torch.uint8), g((ds.n, 3), f32)
    api.gs_neural_fold(ctx, ds, preact)
    api.gs_neural_prepass(ctx, ds, preact, api.make_camera(w.cameras[0]), rgba, color)
    # separate-pass decode of the three models
    for app in (scenes.APP_SH, scenes.APP_NEURAL, scenes.APP_SV):
        sc, dirs, gcol = scenes.config5(4_133, app)
        da = api.upload_scene(sc, dev)
        d = torch.from_numpy(dirs).to(dev); gc = torch.from_numpy(gcol).to(dev)
        col = g((sc.n, 3), f32)
        api.gs_appearance_forward(ctx, da, d, col)
        grads = api.Grads(None, None, None, None, g((sc.n, 3), f32))
        if app == scenes.APP_SH:
            grads.sh_rest = g((sc.n, 15, 3), f32)
        elif app == scenes.APP_SV:
            grads.sv_sites = g((sc.n, 7, 7), f32)
        else:
            grads.features, grads.mlp_weights = g((sc.n, 8), f32), g((816,), f32)
        api.gs_appearance_backward(ctx, da, d, gc, grads, g((sc.n, 3), f32))
    torch.cuda.synchronize()
    api.gs_async_status(ctx)
    g.check()
    ctx.close()
