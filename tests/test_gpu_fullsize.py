"""Checks at the benchmark's full sizes (the launch configuration bench.py times).

The oracle finishes a full-size step of the MLP configuration in seconds, so that one is compared
with it directly.  A full-size ResNet step is minutes of fp64 CPU work, so there the test checks what
holds at any size:
  * the delay schedule observed on the device equals the closed forms of Sec. 3.2 at every step;
  * the two execution modes (one stream per module / one stream for all) give bit-identical weights;
  * rows of (softmax - onehot) sum to zero, so the classifier's bias gradient sums to zero;
  * batch-norm makes the loss invariant to the scale of each output channel of the convolution in
    front of it, so <dW[c], W[c]> = 0 for every such channel (this ties the convolution's weight
    gradient, the batch-norm backward pass and the weights the backward pass read together).
"""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import closed_form_trace, make_ctx, run_parity

pytestmark = pytest.mark.gpu


def test_config2_full_size_against_the_oracle(orc):
    net = sy.config(1)                      # 3072 -> 8 x 1024 -> 10, K = 4, 4 workers x 128
    # lr 0.05 makes this configuration's loss climb from 3 to 7 within a few iterations (an unstable run amplifies
    # every rounding difference), so only the first backward pass is held to 2e-2; later ones to 1e-1
    rec = run_parity(orc, net, 2 * net.K + 2, grad_tol=2e-2, grad_tol_later=1e-1, grad_steps=2 * net.K - 1, loss_tol=1e-2, perturb=False)
    assert not np.isnan(rec[-1]["loss_g"])


def _run(net, p0, steps, serial):
    import torch
    from paper_2509_05679_b200 import binding
    ctx = make_ctx(net, p0, serial=serial)
    xs = [binding.to_device(net.dtype, sy.batch_inputs(net, t)) for t in range(2)]
    ys = [torch.from_numpy(sy.batch_labels(net, t)).cuda() for t in range(2)]
    traces = []
    for t in range(steps):
        ctx.step(xs[t % 2], ys[t % 2])
        f, b, v = ctx.trace()
        traces.append((f.copy(), b.copy(), v.copy()))
    out = ctx.params(), ctx.grads(), traces
    ctx.close()
    return out


def test_config4_full_size_schedule_invariants_and_mode_equivalence():
    net = sy.config(3)                      # ResNet-18-shaped, K = 4, 8 workers x 128: what bench.py times
    p0 = sy.init_params(net.layers, 0, bf16=True)
    steps = 2 * net.K + 1
    params, grads, traces = _run(net, p0, steps, serial=False)
    for t, (f, b, v) in enumerate(traces):
        fc, bc, vc = closed_form_trace(net.K, t)
        assert (f == fc).all() and (b == bc).all() and (v == vc).all(), t
    assert np.isfinite(params).all() and np.isfinite(grads).all()
    # classifier bias gradient sums to zero (fp32 sums of bf16 terms scaled by 1/1024)
    fc_bias = grads[-net.classes:]
    assert abs(fc_bias.sum()) <= 1e-3 * np.abs(fc_bias).sum()
    # scale invariance of every conv that feeds a batch-norm (per layer: |sum_c <dW_c, W_c>| against ||dW|| ||W||)
    off, worst = 0, 0.0
    shapes = sy.param_shapes(net.layers)
    for idx, (li, name, shape, _) in enumerate(shapes):
        n = int(np.prod(shape))
        followed_by_bn = name in ("W", "Wp") and idx + 1 < len(shapes) and shapes[idx + 1][1].startswith("gamma")
        if followed_by_bn and len(shape) == 4:
            w = params[off:off + n].astype(np.float64).reshape(shape[0], -1)
            g = grads[off:off + n].astype(np.float64).reshape(shape[0], -1)
            per_channel = np.abs((w * g).sum(1)) / (np.linalg.norm(w, axis=1) * np.linalg.norm(g, axis=1) + 1e-300)
            worst = max(worst, float(np.median(per_channel)))
            assert np.median(per_channel) <= 2e-2, (li, name, float(np.median(per_channel)))
        off += n
    assert worst > 0
    params_serial, _, _ = _run(net, p0, steps, serial=True)
    assert np.array_equal(params, params_serial)
