"""Parity of gs_adam_step (through the C ABI) against the oracle's Adam step, element by element: the
parameter sets of both appearance models, several steps in a row, ragged sizes, the half-precision
copy, and the argument checks."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

Y0 = 0.28209479177387814
F32 = lambda x: float(np.float32(x))


def _param_sets(n, rng):
    """(name, cols, learning rates, beta2) of the tensors a model trains.  Appearance rates are the
    paper's (App. B, learning-rate table); the geometry rates are the customary ones, which the paper
    leaves to its base method."""
    geo = [("means", 3, [1.6e-4] * 3, 0.999), ("log_scales", 3, [5e-3] * 3, 0.999), ("quats", 4, [1e-3] * 4, 0.999),
           ("opacity_logits", 1, [5e-2], 0.999)]
    sh = geo + [("base_color", 3, [0.0025 * Y0] * 3, 0.999), ("sh_rest", 45, [0.000125] * 45, 0.999)]
    nn = geo + [("base_color", 3, [0.00025] * 3, 0.999), ("features", 8, [0.008] * 8, 0.999),
                ("mlp_weights", 1, [0.003], 0.99)]
    return {"sh": sh, "neural": nn}


def _run_case(oracle, n, model, steps, seed, mixed_lr=False):
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    rng = np.random.default_rng(seed)
    specs = _param_sets(n, rng)[model]
    host, tensors = {}, []
    for name, cols, lr, beta2 in specs:
        rows = 816 if name == "mlp_weights" else n
        if mixed_lr:
            lr = list(np.asarray(lr) * rng.uniform(0.2, 5.0, cols))
        p = rng.normal(0, 1, (rows, cols)).astype(np.float32)
        host[name] = dict(p=p.astype(np.float64), m=np.zeros((rows, cols)), v=np.zeros((rows, cols)), lr=np.asarray(lr, np.float32),
                          beta2=beta2, cols=cols, rows=rows, m_abs=np.zeros((rows, cols)))
        d = {k: torch.from_numpy(a).to(dev) for k, a in (("p", p), ("m", np.zeros_like(p)), ("v", np.zeros_like(p)))}
        d["g"] = torch.empty_like(d["p"])
        d["h"] = torch.full((rows, cols), float("nan"), device=dev, dtype=torch.float16) if name in ("features", "mlp_weights") else None
        host[name]["dev"] = d
        tensors.append(api.AdamTensor(d["p"], d["g"], d["m"], d["v"], host[name]["lr"], 0.9, beta2, 1e-15, half_copy=d["h"]))
    for step in range(1, steps + 1):
        for name, cols, _, _ in specs:
            h = host[name]
            scale = 10.0 ** rng.uniform(-6, 0)                       # gradients of very different sizes
            g = (rng.normal(0, 1, (h["rows"], cols)) * scale).astype(np.float32)
            g[rng.random((h["rows"], cols)) < 0.3] = 0.0               # invisible Gaussians: exact zeros
            h["dev"]["g"].copy_(torch.from_numpy(g))
            # the oracle gets the hyper-parameters as the library does: the fp32 values, widened exactly
            h["p"], h["m"], h["v"] = oracle.adam_step(h["p"], g, h["m"], h["v"], h["lr"].astype(np.float64), F32(0.9),
                                                      F32(h["beta2"]), F32(1e-15), step)
            h["m_abs"] = F32(0.9) * h["m_abs"] + (1 - F32(0.9)) * np.abs(g)    # size of the terms m is made of
        api.gs_adam_step(ctx, tensors, step)
    torch.cuda.synchronize()
    for name, cols, _, _ in specs:
        h, d = host[name], host[name]["dev"]
        p, m, v = (d[k].cpu().numpy().astype(np.float64) for k in ("p", "m", "v"))
        assert np.all(np.abs(m - h["m"]) <= 1e-6 * h["m_abs"] + 1e-37), name       # signed terms may cancel
        assert np.allclose(v, h["v"], rtol=4e-6, atol=1e-37), name
        # the parameter: fp32 rounding of the value itself (6e-8 relative per step) plus 1e-5 of the total movement
        tol = 1e-6 * np.abs(h["p"]) * steps ** 0.5 + 2e-5 * steps * h["lr"][None, :].astype(np.float64)
        assert np.all(np.abs(p - h["p"]) <= tol), (name, np.abs(p - h["p"]).max())
        if d["h"] is not None:                                         # the half copy: RNE of the GPU's own fp32 value
            assert np.array_equal(d["h"].cpu().numpy().view(np.uint16), d["p"].cpu().numpy().astype(np.float16).view(np.uint16))
    ctx.close()


@pytest.mark.parametrize("model", ["sh", "neural"])
def test_adam_matches_oracle_over_several_steps(oracle, model):
    _run_case(oracle, 10_007, model, steps=4, seed=11)        # ragged: 10 007 rows, 45 / 3 / 1 columns


def test_adam_per_column_rates_and_tiny_tensors(oracle):
    _run_case(oracle, 5, "sh", steps=3, seed=12, mixed_lr=True)          # every tensor smaller than one chunk
    _run_case(oracle, 4099, "neural", steps=2, seed=13, mixed_lr=True)


def test_adam_first_step_closed_form_at_full_size():
    """1M rows: after step 1 every element moved by lr_c * g / (|g| + eps), zero gradients not at all -
    a property that holds at any size, checked on every element."""
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    n, cols = 1_000_000, 45
    gen = torch.Generator(device=dev); gen.manual_seed(3)
    p0 = torch.randn((n, cols), device=dev, generator=gen)
    g = torch.randn((n, cols), device=dev, generator=gen) * 1e-3
    g[::7] = 0.0
    lr = np.linspace(1e-4, 2e-3, cols).astype(np.float32)
    p, m, v = p0.clone(), torch.zeros_like(p0), torch.zeros_like(p0)
    api.gs_adam_step(ctx, [api.AdamTensor(p, g, m, v, lr, 0.9, 0.999, 1e-15)], 1)
    torch.cuda.synchronize()
    want = p0.double() - torch.from_numpy(lr.astype(np.float64)).to(dev) * torch.sign(g).double()
    err = (p.double() - want).abs()
    assert float(err.max()) <= 1e-6 * float(p0.abs().max()) + 1e-8
    assert torch.equal(p[::7], p0[::7])
    # the betas are fp32 values: 1 - beta is taken from those
    assert torch.allclose(m.double(), (1 - F32(0.9)) * g.double(), rtol=1e-6, atol=0)
    assert torch.allclose(v.double(), (1 - F32(0.999)) * g.double() ** 2, rtol=1e-6, atol=1e-40)
    ctx.close()


def test_adam_argument_errors():
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    t = lambda: torch.zeros((16, 3), device=dev)
    ok = api.AdamTensor(t(), t(), t(), t(), [1e-3] * 3)
    api.gs_adam_step(ctx, [], 1)                                        # nothing to do is fine
    with pytest.raises(api.GsError) as e:
        api.gs_adam_step(ctx, [ok], 0)
    assert e.value.status == api.GS_ERR_INVALID_ARG
    with pytest.raises(api.GsError):
        api.gs_adam_step(ctx, [ok] * 9, 1)
    bad = api.AdamTensor(t(), t(), t(), t(), [1e-3] * 3, beta2=1.0)
    with pytest.raises(api.GsError):
        api.gs_adam_step(ctx, [bad], 1)
    mis = api.AdamTensor(t().view(-1)[1:4].view(1, 3), t().view(-1)[:3].view(1, 3), t().view(-1)[:3].view(1, 3),
                         t().view(-1)[:3].view(1, 3), [1e-3] * 3)
    with pytest.raises(api.GsError):
        api.gs_adam_step(ctx, [mis], 1)
    torch.cuda.synchronize()
    ctx.close()


def test_adam_sums_the_gradient_buffers_of_several_views(oracle):
    """grad + more_grads[0..6] is the gradient of the step: against the oracle fed with their sum."""
    import torch
    from paper_2609_05255_b200 import api
    ctx = api.Context(0)
    dev = ctx.device
    rng = np.random.default_rng(41)
    rows, cols, views = 3_001, 8, 8
    p0 = rng.normal(size=(rows, cols)).astype(np.float32)
    gs = [(rng.normal(size=(rows, cols)) * 10.0 ** rng.uniform(-4, 0)).astype(np.float32) for _ in range(views)]
    lr = np.full(cols, 0.008, np.float32)
    p, m, v = (torch.from_numpy(a).to(dev) for a in (p0.copy(), np.zeros_like(p0), np.zeros_like(p0)))
    dg = [torch.from_numpy(g).to(dev) for g in gs]
    half = torch.empty((rows, cols), device=dev, dtype=torch.float16)
    t = api.AdamTensor(p, dg[0], m, v, lr, 0.9, 0.999, 1e-15, half_copy=half, more_grads=dg[1:])
    hp, hm, hv = p0.astype(np.float64), np.zeros((rows, cols)), np.zeros((rows, cols))
    for step in (1, 2, 3):
        api.gs_adam_step(ctx, [t], step)
        hp, hm, hv = oracle.adam_step(hp, np.sum([g.astype(np.float64) for g in gs], 0), hm, hv, lr.astype(np.float64),
                                      F32(0.9), F32(0.999), F32(1e-15), step)
    torch.cuda.synchronize()
    # the sum of eight fp32 gradients carries up to 4 ulp of the largest one
    assert np.all(np.abs(p.cpu().numpy() - hp) <= 1e-6 * np.abs(hp) + 1e-4 * 3 * lr[0])
    # v is made of (sum g_k)^2: where the eight terms cancel, the fp32 sum is off by up to 5e-7 of sum |g_k|
    g_sum = np.sum([g.astype(np.float64) for g in gs], 0)
    e_g = 5e-7 * np.sum([np.abs(g).astype(np.float64) for g in gs], 0)
    tol_v = 1e-5 * hv + 3 * (1 - F32(0.999)) * (2 * np.abs(g_sum) * e_g + e_g ** 2)
    assert np.all(np.abs(v.cpu().numpy() - hv) <= tol_v)
    with pytest.raises(api.GsError):
        api.gs_adam_step(ctx, [api.AdamTensor(p, dg[0], m, v, lr, more_grads=dg + dg[:1])], 4)      # nine in all: too many
    ctx.close()
