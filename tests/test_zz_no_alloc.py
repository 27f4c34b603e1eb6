"""The allocation-free entry point gs_appearance_backward_noalloc (collected last on purpose: a run
that stops at the first failure has then already run every other test).

Who needs it: code that cannot call cudaMalloc where it runs - a plugin inside an application that
hands out all device memory at start-up, a real-time loop that may not stall on the allocator, or a
caller that cannot create a GsContext (gs_create allocates).  The library keeps the kernel's scratch
(partial sums of the decoder-weight gradient) in a static device array instead.

The test calls it through the C ABI twice in a row, with different sizes and data, and checks every
output against gs_appearance_backward on the same inputs.
"""
import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import grad_mismatch

pytestmark = pytest.mark.gpu


def _inputs(n, seed, device):
    import torch
    from paper_2609_05255_b200 import api
    sc, dirs, gcol = scenes.config5(n, scenes.APP_NEURAL)
    rng = np.random.default_rng(seed)
    sc.features = rng.normal(0, 0.3, sc.features.shape).astype(np.float16)     # differ between the calls
    gcol = rng.standard_normal(gcol.shape).astype(np.float32)
    ds = api.upload_scene(sc, device)
    return ds, torch.from_numpy(dirs).to(device), torch.from_numpy(gcol).to(device)


def test_noalloc_matches_the_allocating_entry_point_twice_in_a_row():
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)                       # only the existing entry point needs a context
    api.gs_set_decoder_engine(ctx, api.GS_ENGINE_WARP_MMA)   # the kernel the allocation-free entry point runs
    dev = ctx.device
    # second call smaller than the first: rows of the shared scratch left over from call 1 must not leak
    for n, seed in ((70_001, 1), (9_000, 2)):
        ds, dirs, gcol = _inputs(n, seed, dev)
        want = api.alloc_grads(n, api.GS_APP_NEURAL, dev); want_d = torch.empty((n, 3), device=dev)
        got = api.alloc_grads(n, api.GS_APP_NEURAL, dev); got_d = torch.full((n, 3), float("nan"), device=dev)
        got.mlp_weights.fill_(float("nan")); got.features.fill_(float("nan")); got.base_color.fill_(float("nan"))
        api.gs_appearance_backward(ctx, ds, dirs, gcol, want, want_d)
        torch.cuda.synchronize()
        # free device memory as the driver reports it (cudaMemGetInfo): an allocation made inside the library would
        # show here, which torch's own counters cannot see.  The first call on a device may load the library's
        # module, so the figure is taken around a repeated call.
        api.gs_appearance_backward_noalloc(ds, dirs, gcol, got, got_d)
        torch.cuda.synchronize()
        before = torch.cuda.mem_get_info(dev)[0]
        api.gs_appearance_backward_noalloc(ds, dirs, gcol, got, got_d)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(dev)[0] == before
        # per-Gaussian outputs come from the same kernel code: identical bits
        assert torch.equal(got.base_color, want.base_color)
        assert torch.equal(got.features, want.features)
        assert torch.equal(got_d, want_d)
        # the weight gradient is the same sum in another order: the tolerance the other tests use for
        # the 816 weight gradients (1e-3 relative or 1e-5 absolute, for all but 2 % of them: each sums
        # tens of thousands of signed terms, so a few cancel to well below the size of their terms),
        # and no element off by more than 1e-4 of the largest one
        w_got, w_want = got.mlp_weights.cpu().numpy(), want.mlp_weights.cpu().numpy()
        assert np.all(np.isfinite(w_got)) and np.abs(w_want).max() > 1
        assert grad_mismatch(w_got, w_want).mean() <= 0.02
        assert np.abs(w_got - w_want).max() <= 1e-4 * np.abs(w_want).max()
    ctx.close()


def test_noalloc_rejects_what_it_cannot_serve():
    import torch
    from paper_2609_05255_b200 import api
    dev = torch.device("cuda", 0)
    ds, dirs, gcol = _inputs(256, 3, dev)
    grads = api.alloc_grads(256, api.GS_APP_NEURAL, dev); gd = torch.empty((256, 3), device=dev)
    grads.mlp_weights.fill_(7.0)
    cs = ds.c_struct()
    cs.n = api.NOALLOC_MAX_N + 1               # only the size is checked before the refusal: nothing is read
    import ctypes as C
    msg = C.create_string_buffer(256)
    st = api._lib.gs_appearance_backward_noalloc(C.byref(cs), dirs.data_ptr(), gcol.data_ptr(),
                                                 C.byref(grads.c_struct()), gd.data_ptr(), None, msg, len(msg))
    assert st == api.GS_ERR_CAPACITY and b"4194304" in msg.value
    torch.cuda.synchronize()
    assert torch.all(grads.mlp_weights == 7.0)  # nothing was launched
    ds.app = api.GS_APP_SH
    with pytest.raises(api.GsError) as e:
        api.gs_appearance_backward_noalloc(ds, dirs, gcol, grads, gd)
    assert e.value.status == api.GS_ERR_UNSUPPORTED
    ds.app = api.GS_APP_NEURAL
    for field, value in (("color_activation", 9), ("decoder_precision", 5)):
        old = getattr(ds, field)
        setattr(ds, field, value)
        with pytest.raises(api.GsError) as e:
            api.gs_appearance_backward_noalloc(ds, dirs, gcol, grads, gd)
        assert e.value.status == api.GS_ERR_INVALID_ARG, field
        setattr(ds, field, old)
    torch.cuda.synchronize()
    assert torch.all(grads.mlp_weights == 7.0)


def test_noalloc_honours_the_decoder_precision_and_the_colour_activation():
    """The two scene fields that select another instance of the kernel: results must equal those of the allocating
    entry point given the same fields."""
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    api.gs_set_decoder_engine(ctx, api.GS_ENGINE_WARP_MMA)
    dev = ctx.device
    n = 33_333
    ds, dirs, gcol = _inputs(n, 4, dev)
    for precision, act in ((api.GS_DECODER_HALF, 0), (api.GS_DECODER_SPLIT, 2)):
        ds.decoder_precision = precision; ds.color_activation = act
        want = api.alloc_grads(n, api.GS_APP_NEURAL, dev); want_d = torch.empty((n, 3), device=dev)
        got = api.alloc_grads(n, api.GS_APP_NEURAL, dev); got_d = torch.empty((n, 3), device=dev)
        api.gs_appearance_backward(ctx, ds, dirs, gcol, want, want_d)
        api.gs_appearance_backward_noalloc(ds, dirs, gcol, got, got_d)
        torch.cuda.synchronize()
        assert torch.equal(got.base_color, want.base_color) and torch.equal(got.features, want.features)
        assert torch.equal(got_d, want_d)
        w_got, w_want = got.mlp_weights.cpu().numpy(), want.mlp_weights.cpu().numpy()
        assert np.abs(w_got - w_want).max() <= 1e-4 * np.abs(w_want).max()
    # the unsplit kernel is a different computation: its features gradient differs from the split one's
    ds.decoder_precision = api.GS_DECODER_SPLIT; ds.color_activation = 0
    split = api.alloc_grads(n, api.GS_APP_NEURAL, dev); sd = torch.empty((n, 3), device=dev)
    api.gs_appearance_backward_noalloc(ds, dirs, gcol, split, sd)
    ds.decoder_precision = api.GS_DECODER_HALF
    half = api.alloc_grads(n, api.GS_APP_NEURAL, dev)
    api.gs_appearance_backward_noalloc(ds, dirs, gcol, half, sd)
    torch.cuda.synchronize()
    assert not torch.equal(split.features, half.features)
    ctx.close()
