"""Parity at the full benchmark sizes, in the launch configuration bench.py times: the 100k-Gaussian
512x512 scene, one view of the 1M-Gaussian 1256x828 scene (neural and SH) and one view of the
3M-Gaussian 1920x1080 scene (config 1 runs at its full size among the small cases), checked
against the oracle with the same stage-by-stage rules as the small cases."""
from types import SimpleNamespace

import numpy as np
import pytest

from paper_2609_05255_b200 import scenes
from gpu_helpers import run_gpu
import test_gpu_parity as small

pytestmark = pytest.mark.gpu

CASES = {
    "config2_neural_100k": lambda: (scenes.config2(), 0),
    "config3_neural_1M": lambda: (scenes.config3(scenes.APP_NEURAL), 2),
    "config3_sh_1M": lambda: (scenes.config3(scenes.APP_SH), 5),
    "config3_sv_1M": lambda: (scenes.config3(scenes.APP_SV), 1),
    "config4_neural_3M": lambda: (scenes.config4(), 7),
}


@pytest.fixture(scope="module", params=list(CASES))
def full(request, oracle):
    w, view = CASES[request.param]()
    cam = w.cameras[view]
    G = scenes.upstream_gradient(cam, 777)
    gpu = run_gpu(w.scene, cam, G)
    fwd, grads = oracle.render(w.scene, cam, G, with_abs=False)
    m2, co, col = (a.astype(np.float64) for a in (gpu.mean2d, gpu.conic_opacity, gpu.color))
    for a in (m2, co, col):
        a[~gpu.visible] = 0
    iso = oracle.blend_forward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col)
    iso_g = oracle.blend_backward(cam, gpu.sorted_vals, gpu.tile_ranges, m2, co[:, :3], co[:, 3], col, G,
                                  with_abs=True)
    r = SimpleNamespace(w=w, cam=cam, G=G, gpu=gpu, fwd=fwd, grads=grads, iso=iso, iso_g=iso_g)
    return {request.param: r}, request.param


def test_full_size_per_gaussian_floats(full):
    results, name = full
    small.test_per_gaussian_floats(results, name)


def test_full_size_integer_stage_bit_exact(full, oracle):
    results, name = full
    small.test_integer_stage_bit_exact(results, oracle, name)


def test_full_size_image(full):
    results, name = full
    small.test_image(results, name)


def test_full_size_blend_backward(full):
    results, name = full
    small.test_blend_backward_2d_gradients(results, name)


def test_full_size_parameter_gradients(full, oracle):
    results, name = full
    small.test_parameter_gradients(results, oracle, name)
