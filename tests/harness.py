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
    """Per tensor: max_i |a_i - b_i| / max(|b_i|, 0.1 * rms(b)); returns the worst tensor.
    The floor exists because an fp32 sum of terms of size s carries an absolute error of about
    2^-24 * s however small the sum itself turns out (cancellation): an element far below the
    tensor's scale cannot be held to a RELATIVE 1e-5 by any fp32 evaluation order."""
    worst, where = 0.0, ""
    for name, sl in tensor_slices(layers):
        bb, aa = np.asarray(b[sl], np.float64), np.asarray(a[sl], np.float64)
        floor = 0.1 * np.sqrt(np.mean(bb * bb)) + 1e-30
        e = float(np.max(np.abs(aa - bb) / np.maximum(np.abs(bb), floor)))
        if e > worst:
            worst, where = e, name
    return worst, where


def grad_rel_l2(a, b, layers, min_norm=1e-12):
    """Per tensor ||a - b||_2 / ||b||_2 (tensors whose reference gradient is ~0 are skipped).
    Returns (worst error, its tensor, {tensor: error})."""
    worst, where, per = 0.0, "", {}
    for name, sl in tensor_slices(layers):
        bb, aa = np.asarray(b[sl], np.float64), np.asarray(a[sl], np.float64)
        nb = np.linalg.norm(bb)
        if nb < min_norm:
            continue
        e = float(np.linalg.norm(aa - bb) / nb)
        per[name] = e
        if e > worst:
            worst, where = e, name
    return worst, where, per


def make_oracle(orc, net: sy.Net, params, storage_model=True):
    """The oracle for a configuration; bf16 configurations get the bf16 storage model."""
    o = orc.Oracle(net.layers, net.splits, net.n_workers, net.batch, (net.in_h, net.in_w, net.in_c), net.classes)
    o.storage_bf16(storage_model and net.dtype == "bf16")
    o.set_params(params)
    return o


def make_ctx(net: sy.Net, params, **kw):
    from paper_2509_05679_b200 import binding
    ctx = binding.Context(net.layers, net.splits, net.n_workers, net.batch, net.lr, dtype=net.dtype,
                          in_shape=(net.in_h, net.in_w, net.in_c), num_classes=net.classes, **kw)
    ctx.set_params(params)
    return ctx


def pick_data_stream(orc, net: sy.Net, p0, steps: int, guard: float, tries: int = 16) -> int:
    """First data stream for which, in the ORACLE's run, no ReLU input and no max-pool top-2 gap
    ever comes closer to its kink than `guard`.  Tight fp32 tolerances only make sense on such
    a run: nearer to a kink, fp32 and fp64 may legitimately take different branches.  The choice
    is made by the oracle alone, before the library runs."""
    for stream in range(tries):
        o = make_oracle(orc, net, p0)
        orc.kink_margin(True)
        for t in range(steps):
            o.step(sy.batch_inputs(net, t, stream), sy.batch_labels(net, t, stream), net.lr)
        if orc.kink_margin(True) >= guard:
            return stream
    raise AssertionError("no data stream keeps every pre-activation away from the kinks")


def module_bounds(net):
    return [0] + list(net.splits) + [len(net.layers)]


def closed_form_trace(K, t):
    f = np.array([t - k + 1 if t - k + 1 >= 0 else -1 for k in range(1, K + 1)])
    b = np.array([t - 2 * K + k + 1 if t - 2 * K + k + 1 >= 0 else -1 for k in range(1, K + 1)])
    v = np.array([t - 2 * K + 2 * k if t - 2 * K + k + 1 >= 0 else -1 for k in range(1, K + 1)])
    return f, b, v


def run_parity(orc, net: sy.Net, steps: int, *, param_tol=None, grad_tol=None, grad_best_tol=None, loss_tol=None,
               perturb=True, kink_guard=None, grad_steps=None, grad_tail=None, grad_tol_later=None, **ctx_kw):
    """Step both implementations `steps` times; check the schedule bit-exactly after every step and
    parameters / gradients / loss within the given tolerances.  Returns the per-step records.

    Gradients: every tensor must be within `grad_tol` at every step.  `grad_best_tol` is a much
    tighter bound on each tensor's BEST step: a pre-activation that lands on the other side of a
    ReLU / max-pool kink in one precision but not the other legitimately changes a few terms of a
    gradient sum in that step, whereas a wrong formula is wrong at every step.
    `grad_steps`: check gradients only while t < grad_steps (afterwards the two trajectories have
    moved apart and a gradient comparison compares different weights).  `grad_tail`: hold only the
    last `grad_tail` tensors to `grad_tol` and ask the whole gradient for a cosine similarity of 0.7
    (deep batch-norm networks amplify a single rounding difference by orders of magnitude on the
    way back to the first layers).  `grad_tol_later`: tolerance after the run's first backward pass
    (t = K-1, held to `grad_tol`): from then on the weights of the two runs differ by their
    earlier gradient differences."""
    from paper_2509_05679_b200 import binding
    bf16 = net.dtype == "bf16"
    p0 = sy.init_params(net.layers, 0, bf16=False)
    if perturb:
        p0 = sy.perturb_params(p0, net.layers, 7, 0.1)
    if bf16:
        p0 = sy.round_to_bf16(p0)
    stream = pick_data_stream(orc, net, p0, steps, kink_guard) if kink_guard else 0
    o = make_oracle(orc, net, p0)
    ctx = make_ctx(net, p0, **ctx_kw)
    rec, best = [], {}
    try:
        for t in range(steps):
            x, y = sy.batch_inputs(net, t, stream), sy.batch_labels(net, t, stream)
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
            if grad_tol is not None and (grad_steps is None or t < grad_steps):
                g_avg = np.mean([o.grads(s) for s in range(net.n_workers)], axis=0)     # P = 11^T/N averages the workers
                g_gpu = ctx.grads()
                r["grad_err"], r["grad_where"], per = grad_rel_l2(g_gpu, g_avg, net.layers)
                for k_, e_ in per.items():
                    best[k_] = min(best.get(k_, np.inf), e_)
                if grad_tail is None and grad_tol_later is None:
                    assert r["grad_err"] <= grad_tol, (t, r)
                elif grad_tail is None:
                    first = t == net.K - 1          # the first backward pass of the run: no weight has changed yet
                    assert r["grad_err"] <= (grad_tol if first else grad_tol_later), (t, r)
                elif per:
                    tail = list(per.items())[-grad_tail:]
                    assert all(e_ <= grad_tol for _, e_ in tail), (t, tail)
                    nz = np.abs(g_avg) > 0
                    cos = float(np.dot(g_gpu[nz], g_avg[nz]) / (np.linalg.norm(g_gpu[nz]) * np.linalg.norm(g_avg[nz]) + 1e-300))
                    r["grad_cos"] = cos
                    assert cos >= 0.7, (t, cos)
            if param_tol is not None:
                r["param_err"], r["param_where"] = max_rel_err(ctx.params(), o.params(0), net.layers)
                assert r["param_err"] <= param_tol, (t, r)
            rec.append(r)
    finally:
        ctx.close()
    if grad_best_tol is not None:
        assert best and len(best) == len(tensor_slices(net.layers)), "some tensor never received a gradient"
        bad = {k_: e_ for k_, e_ in best.items() if e_ > grad_best_tol}
        assert not bad, bad
    return rec
