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


FP32_FLOOR = 0.1           # of the tensor's rms


def max_rel_err(a, b, layers):
    """Per tensor: max_i |a_i - b_i| / max(|b_i|, 0.1 * rms(b)); returns the worst tensor.
    The floor exists because an fp32 sum of terms of size s carries an absolute error of a few
    2^-24 * s however small the sum itself turns out (cancellation), and a parameter collects one such
    error per update: an element far below its tensor's scale cannot be held to a RELATIVE 1e-5 by any
    fp32 evaluation order.  Measured over the fp32 tests of this directory (B200): the worst element is
    off by 2.2e-7 of its tensor's rms after one update and by 6.1e-7 after 10-18 updates (ten fp32 ulps of
    an rms-sized value), which is 1.2e-5 against a floor of 0.05 rms and 6e-6 against this one."""
    worst, where = 0.0, ""
    for name, sl in tensor_slices(layers):
        bb, aa = np.asarray(b[sl], np.float64), np.asarray(a[sl], np.float64)
        floor = FP32_FLOOR * np.sqrt(np.mean(bb * bb)) + 1e-30
        e = float(np.max(np.abs(aa - bb) / np.maximum(np.abs(bb), floor)))
        if e > worst:
            worst, where = e, name
    return worst, where


def gradient_groups(layers, pair_bn=False):
    """[(name, index array)] of the tensors a gradient comparison looks at.  pair_bn (networks without ReLU layers): the
    tensors of one layer form one group (W with b, gamma with beta, a projection's W with its gamma and beta).  There a
    shift of a layer's output is removed again by the next batch-norm, so the gradient of a bias or a beta that only feeds
    batch-normed paths is what the zero padding at the image border leaves of it, tens of times smaller than its layer's
    other gradient and no scale to measure an error against."""
    sl = tensor_slices(layers)
    if not pair_bn:
        return [(name, np.r_[s]) for name, s in sl]
    out = []
    for name, s in sl:
        layer = name.split(".")[0]
        if out and out[-1][0].split(".")[0] == layer:
            out[-1] = (out[-1][0] + "+" + name.split(".")[1], np.r_[out[-1][1], s])
        else:
            out.append((name, np.r_[s]))
    return out


def grad_rel_l2(a, b, layers, min_norm=1e-12, pair_bn=False):
    """Per tensor ||a - b||_2 / ||b||_2 (tensors whose reference gradient is ~0 are skipped).
    Returns (worst error, its tensor, {tensor: error})."""
    worst, where, per = 0.0, "", {}
    for name, ix in gradient_groups(layers, pair_bn):
        bb, aa = np.asarray(b[ix], np.float64), np.asarray(a[ix], np.float64)
        nb = np.linalg.norm(bb)
        if nb < min_norm:
            continue
        e = float(np.linalg.norm(aa - bb) / nb)
        per[name] = e
        if e > worst:
            worst, where = e, name
    return worst, where, per


def grad_max_err(a, b, layers, min_norm=1e-12, pair_bn=False):
    """Element by element: per tensor max_i |a_i - b_i| / max_i |b_i|.  Returns (worst, its tensor)."""
    worst, where = 0.0, ""
    for name, ix in gradient_groups(layers, pair_bn):
        bb, aa = np.asarray(b[ix], np.float64), np.asarray(a[ix], np.float64)
        if np.linalg.norm(bb) < min_norm:
            continue
        e = float(np.max(np.abs(aa - bb)) / np.max(np.abs(bb)))
        if e > worst:
            worst, where = e, name
    return worst, where


def ulp_perturbed(x, fraction=1e-3, seed=5):
    """A copy of a bf16-representable array with `fraction` of its values moved to the next bf16 value away
    from zero: the smallest change of the inputs a bf16 run can see."""
    g = np.random.Generator(np.random.Philox(key=seed))
    flat = np.ascontiguousarray(x, dtype=np.float32).reshape(-1).copy()
    idx = g.choice(flat.size, max(1, int(fraction * flat.size)), replace=False)
    flat[idx] = (flat[idx].view(np.uint32) + np.uint32(0x10000)).view(np.float32)
    return flat.reshape(x.shape)


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
               perturb=True, kink_guard=None, grad_steps=None, grad_tol_later=None, elem_tol=None, pair_bn=False,
               noise_factor=None, elem_noise_factor=None, **ctx_kw):
    """Step both implementations `steps` times; check the schedule bit-exactly after every step and
    parameters / gradients / loss within the given tolerances.  Returns the per-step records.

    Gradients: every tensor must be within `grad_tol` (relative L2) at every step, and, with `elem_tol`,
    every element within `elem_tol` of the tensor's largest element.  `grad_best_tol` is a much
    tighter bound on each tensor's BEST step: a pre-activation that lands on the other side of a
    ReLU / max-pool kink in one precision but not the other legitimately changes a few terms of a
    gradient sum in that step, whereas a wrong formula is wrong at every step.
    `grad_steps`: check gradients only while t < grad_steps.  `grad_tol_later`: tolerance after the run's
    first backward pass (t = K-1, held to `grad_tol`): from then on the weights of the two runs differ by
    their earlier gradient differences.
    `noise_factor` (bf16 networks with ReLU layers, where two bf16 evaluations of the same gradient differ by
    tens of percent, see tests/test_oracle_pins.py): a second oracle runs beside the first on inputs of which
    0.1 % were moved by one bf16 ulp; a tensor may deviate from the oracle by `grad_tol` or by `noise_factor`
    times what that twin deviates, whichever is larger (`elem_noise_factor`: the same for the element-wise
    bound `elem_tol`)."""
    from paper_2509_05679_b200 import binding
    import torch
    bf16 = net.dtype == "bf16"
    p0 = sy.init_params(net.layers, 0, bf16=False)
    if perturb:
        p0 = sy.perturb_params(p0, net.layers, 7, 0.1)
    if bf16:
        p0 = sy.round_to_bf16(p0)
    stream = pick_data_stream(orc, net, p0, steps, kink_guard) if kink_guard else 0
    if kink_guard:
        print(f"{net.name}: data stream {stream} keeps every pre-activation {kink_guard:g} away from the kinks")
    o = make_oracle(orc, net, p0)
    twin = make_oracle(orc, net, p0) if noise_factor else None
    ctx = make_ctx(net, p0, **ctx_kw)
    rec, best = [], {}
    try:
        for t in range(steps):
            x, y = sy.batch_inputs(net, t, stream), sy.batch_labels(net, t, stream)
            lo, _ = o.step(x, y, net.lr)
            lg = ctx.step(binding.to_device(net.dtype, x), torch.from_numpy(y).cuda(), want_loss=True)
            fo, bo, vo, _ = o.trace()
            fg, bg, vg = ctx.trace()
            assert (fg == fo).all() and (bg == bo).all() and (vg == vo).all(), (t, fg, fo, bg, bo, vg, vo)
            fc, bc, vc = closed_form_trace(net.K, t)
            assert (fg == fc).all() and (bg == bc).all() and (vg == vc).all()
            r = {"t": t, "loss_o": lo, "loss_g": lg, "stream": stream}
            if np.isnan(lo):
                assert np.isnan(lg)
            elif loss_tol is not None:
                assert abs(lg - lo) <= loss_tol * max(abs(lo), 1e-6), (t, lg, lo)
            if twin is not None:
                twin.step(ulp_perturbed(x, 1e-3, 5 + t), y, net.lr)
            if grad_tol is not None and (grad_steps is None or t < grad_steps):
                g_avg = np.mean([o.grads(s) for s in range(net.n_workers)], axis=0)     # P = 11^T/N averages the workers
                g_gpu = ctx.grads()
                r["grad_err"], r["grad_where"], per = grad_rel_l2(g_gpu, g_avg, net.layers, pair_bn=pair_bn)
                for k_, e_ in per.items():
                    best[k_] = min(best.get(k_, np.inf), e_)
                tol = grad_tol if (grad_tol_later is None or t == net.K - 1) else grad_tol_later
                if twin is None:
                    assert r["grad_err"] <= tol, (t, r)
                else:
                    g_twin = np.mean([twin.grads(s) for s in range(net.n_workers)], axis=0)
                    _, _, noise = grad_rel_l2(g_twin, g_avg, net.layers, pair_bn=pair_bn)
                    bad = {k_: (e_, noise.get(k_, 0.0)) for k_, e_ in per.items() if e_ > max(tol, noise_factor * noise.get(k_, 0.0))}
                    r["noise_max"] = max(noise.values()) if noise else 0.0
                    assert not bad, (t, bad)
                if elem_tol is not None:
                    r["elem_err"], r["elem_where"] = grad_max_err(g_gpu, g_avg, net.layers, pair_bn=pair_bn)
                    bound = elem_tol
                    if twin is not None and elem_noise_factor:
                        r["elem_noise"] = grad_max_err(g_twin, g_avg, net.layers, pair_bn=pair_bn)[0]
                        bound = max(elem_tol, elem_noise_factor * r["elem_noise"])
                    assert r["elem_err"] <= bound, (t, r)
            if param_tol is not None:
                r["param_err"], r["param_where"] = max_rel_err(ctx.params(), o.params(0), net.layers)
                assert r["param_err"] <= param_tol, (t, r)
            rec.append(r)
    finally:
        ctx.close()
    if grad_best_tol is not None:
        assert best and len(best) == len(gradient_groups(net.layers, pair_bn)), "some tensor never received a gradient"
        bad = {k_: e_ for k_, e_ in best.items() if e_ > grad_best_tol}
        assert not bad, bad
    return rec
