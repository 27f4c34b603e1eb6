"""The seeded input generators: determinism, shapes, dtypes and the stated distributions."""
import numpy as np

from paper_2609_05255_b200 import scenes


def test_config1_is_deterministic_and_shaped():
    a, b = scenes.config1(), scenes.config1()
    s = a.scene
    assert s.n == 1000 and s.app == scenes.APP_SH and s.active_degree == 3
    for name in ("means", "log_scales", "quats", "opacity_logits", "base_color", "sh_rest"):
        x, y = getattr(s, name), getattr(b.scene, name)
        assert x.dtype == np.float32 and x.flags.c_contiguous and np.array_equal(x, y)
    assert s.sh_rest.shape == (1000, 15, 3) and s.quats.shape == (1000, 4)
    assert s.means[:, 2].min() >= 2 and s.means[:, 2].max() <= 4 and np.abs(s.means[:, :2]).max() <= 1
    assert abs(s.log_scales.mean() + 3) < 0.05 and abs(s.log_scales.std() - 0.5) < 0.05
    cam = a.cameras[0]
    assert (cam.width, cam.height, cam.fx, cam.cx) == (64, 64, 64.0, 32.0)


def test_neural_appearance_storage():
    w = scenes.config2(n=2000)
    s = w.scene
    assert s.features.dtype == np.float16 and s.features.shape == (2000, 8)
    assert s.mlp_weights.dtype == np.float16 and s.mlp_weights.shape == (816,)
    assert s.base_color.nbytes // 2000 + s.features.nbytes // 2000 == 28
    assert np.abs(s.mlp_weights[:512].astype(np.float32)).max() <= np.sqrt(6 / 48) + 1e-3
    sh = scenes.config2(n=2000, app=scenes.APP_SH).scene
    assert (sh.base_color.nbytes + sh.sh_rest.nbytes) // 2000 == 192


def test_orbit_cameras_look_at_origin():
    cams = scenes.orbit_cameras(1256, 828, 8)
    assert len(cams) == 8
    for c in cams:
        R, t = c.w2c[:, :3].astype(np.float64), c.w2c[:, 3].astype(np.float64)
        assert np.abs(R @ R.T - np.eye(3)).max() < 1e-6 and abs(np.linalg.det(R) - 1) < 1e-6
        origin_cam = t                      # world origin in camera coordinates
        assert np.allclose(origin_cam, [0, 0, 5], atol=1e-5)
        assert abs(c.fx - 628 / np.tan(np.radians(30))) < 1e-2


def test_clustered_scene_statistics():
    s = scenes.clustered_scene(20000, 64, -4.0, 0.7, scenes.APP_SH, seed=1003)
    r = np.linalg.norm(s.means, axis=1)
    shell = np.abs(r - 20) < 1e-3
    assert abs(shell.mean() - 0.1) < 1e-3
    assert np.percentile(r[~shell], 99) < 5
    assert abs(s.opacity_logits.std() - 1.5) < 0.05
