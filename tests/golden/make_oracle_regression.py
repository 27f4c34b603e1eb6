"""Writes tests/golden/oracle_regression.txt: summary numbers of the oracle's own output on small seeded
scenes (all three appearance models, forward and backward, one Adam step, the viewer prepass).  The file is
not a pin of the oracle against the paper - the pins are in tests/test_oracle_*.py - but a guard: a change
to the oracle's arithmetic shows up as a diff of this file and has to be justified where it is made.

Run from the repository root:  python tests/golden/make_oracle_regression.py
Calls only oracle/ and the seeded input generators."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import gs_oracle as oracle          # noqa: E402
from paper_2609_05255_b200 import scenes        # noqa: E402


def summary():
    out = {}
    for tag, w in (("config1_sh", scenes.config1()),
                   ("config2_neural_2000", scenes.config2(n=2000)),
                   ("config2_sv_2000", scenes.config2(n=2000, app=scenes.APP_SV))):
        cam = w.cameras[0]
        G = scenes.upstream_gradient(cam, 4242)
        fwd, g = oracle.render(w.scene, cam, G)
        out[f"{tag}.pairs"] = float(fwd.P)
        out[f"{tag}.image_sum"] = float(fwd.image.sum())
        out[f"{tag}.image_sq"] = float((fwd.image ** 2).sum())
        out[f"{tag}.final_T_sum"] = float(fwd.final_T.sum())
        out[f"{tag}.n_contrib_sum"] = float(fwd.n_contrib.astype(np.int64).sum())
        out[f"{tag}.order_hash"] = float((fwd.vals.astype(np.int64) * (np.arange(len(fwd.vals)) % 9973 + 1)).sum() % 1000003)
        for nm in ("means", "log_scales", "quats", "opacity_logits", "base_color", "sh_rest", "features", "mlp_weights", "sv_sites"):
            a = getattr(g, nm, None)
            if a is not None:
                out[f"{tag}.grad_{nm}_l1"] = float(np.abs(a).sum())
    rng = np.random.default_rng(7)
    p, gr = rng.normal(size=(50, 4)), rng.normal(size=(50, 4))
    p1, m1, v1 = oracle.adam_step(p, gr, 0.1 * gr, 0.01 * gr * gr, np.array([1e-3, 2e-3, 3e-3, 4e-3]), 0.9, 0.99, 1e-8, step=3)
    out["adam.param_sum"] = float(p1.sum()); out["adam.m_sum"] = float(m1.sum()); out["adam.v_sum"] = float(v1.sum())
    sc = scenes.config2(n=500).scene
    pre = oracle.neural_fold(sc)
    out["prepass.pre_l1"] = float(np.abs(pre).sum())
    out["prepass.colour_sum"] = float(oracle.neural_prepass(sc, pre, np.array([0.1, -0.2, -1.0])).sum())
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_regression.txt")
    with open(path, "w") as f:
        f.write("# written by tests/golden/make_oracle_regression.py from the oracle alone; name = value\n")
        for k, v in summary().items():
            f.write(f"{k} = {v!r}\n")
    print("wrote", path)
