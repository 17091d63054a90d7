"""Shared helpers of the GPU parity tests: run the oracle and the library on the same seeded
inputs and compare them (the oracle lives in oracle/, the library behind paper_2509_05679_b200.binding)."""
from __future__ import annotations

import numpy as np

from paper_2509_05679_b200 import synth as sy


def tensor_slices(layers):
    out, off = [], 0
    for li, name, shape, _ in sy.param_shapes(layers):
        n = int(np.prod(shape))
        out.append((f"L{li}.{name}", slice(off, off + n)))
        off += n
    return out


def max_rel_err(a, b, layers):
    """Per tensor: max_i |a_i - b_i| / max(|b_i|, 1e-3 * rms(b)); returns the worst tensor."""
    worst, where = 0.0, ""
    for name, sl in tensor_slices(layers):
        bb, aa = np.asarray(b[sl], np.float64), np.asarray(a[sl], np.float64)
        floor = 1e-3 * np.sqrt(np.mean(bb * bb)) + 1e-30
        e = float(np.max(np.abs(aa - bb) / np.maximum(np.abs(bb), floor)))
        if e > worst:
            worst, where = e, name
    return worst, where


def grad_rel_l2(a, b, layers, min_norm=1e-12):
    """Per tensor ||a - b||_2 / ||b||_2 (tensors whose reference gradient is ~0 are skipped)."""
    worst, where = 0.0, ""
    for name, sl in tensor_slices(layers):
        bb, aa = np.asarray(b[sl], np.float64), np.asarray(a[sl], np.float64)
        nb = np.linalg.norm(bb)
        if nb < min_norm:
            continue
        e = float(np.linalg.norm(aa - bb) / nb)
        if e > worst:
            worst, where = e, name
    return worst, where


def make_oracle(orc, net: sy.Net, params):
    o = orc.Oracle(net.layers, net.splits, net.n_workers, net.batch, (net.in_h, net.in_w, net.in_c), net.classes)
    o.set_params(params)
    return o


def make_ctx(net: sy.Net, params, **kw):
    from paper_2509_05679_b200 import binding
    ctx = binding.Context(net.layers, net.splits, net.n_workers, net.batch, net.lr, dtype=net.dtype,
                          in_shape=(net.in_h, net.in_w, net.in_c), num_classes=net.classes, **kw)
    ctx.set_params(params)
    return ctx


def closed_form_trace(K, t):
    f = np.array([t - k + 1 if t - k + 1 >= 0 else -1 for k in range(1, K + 1)])
    b = np.array([t - 2 * K + k + 1 if t - 2 * K + k + 1 >= 0 else -1 for k in range(1, K + 1)])
    v = np.array([t - 2 * K + 2 * k if t - 2 * K + k + 1 >= 0 else -1 for k in range(1, K + 1)])
    return f, b, v


def run_parity(orc, net: sy.Net, steps: int, *, param_tol=None, grad_tol=None, loss_tol=None, perturb=True, **ctx_kw):
    """Step both implementations `steps` times; check the schedule bit-exactly after every step and
    parameters / gradients / loss within the given tolerances.  Returns the per-step records."""
    from paper_2509_05679_b200 import binding
    bf16 = net.dtype == "bf16"
    p0 = sy.init_params(net.layers, 0, bf16=False)
    if perturb:
        p0 = sy.perturb_params(p0, net.layers, 7, 0.1)
    if bf16:
        p0 = sy.round_to_bf16(p0)
    o = make_oracle(orc, net, p0)
    ctx = make_ctx(net, p0, **ctx_kw)
    rec = []
    try:
        for t in range(steps):
            x, y = sy.batch_inputs(net, t), sy.batch_labels(net, t)
            lo, _ = o.step(x, y, net.lr)
            import torch
            lg = ctx.step(binding.to_device(net.dtype, x), torch.from_numpy(y).cuda(), want_loss=True)
            fo, bo, vo, _ = o.trace()
            fg, bg, vg = ctx.trace()
            assert (fg == fo).all() and (bg == bo).all() and (vg == vo).all(), (t, fg, fo, bg, bo, vg, vo)
            fc, bc, vc = closed_form_trace(net.K, t)
            assert (fg == fc).all() and (bg == bc).all() and (vg == vc).all()
            r = {"t": t, "loss_o": lo, "loss_g": lg}
            if np.isnan(lo):
                assert np.isnan(lg)
            elif loss_tol is not None:
                assert abs(lg - lo) <= loss_tol * max(abs(lo), 1e-6), (t, lg, lo)
            if grad_tol is not None:
                r["grad_err"], r["grad_where"] = grad_rel_l2(ctx.grads(), o.grads(0), net.layers)
                assert r["grad_err"] <= grad_tol, (t, r)
            if param_tol is not None:
                r["param_err"], r["param_where"] = max_rel_err(ctx.params(), o.params(0), net.layers)
                assert r["param_err"] <= param_tol, (t, r)
            rec.append(r)
    finally:
        ctx.close()
    return rec
