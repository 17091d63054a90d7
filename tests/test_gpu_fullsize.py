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
import os

import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import closed_form_trace, make_ctx, run_parity

pytestmark = pytest.mark.gpu
# Runs whose oracle side takes several minutes (full-size configuration 2 for its 200 iterations, full-width configuration 3
# for 50) are run on request: FDG_LONG_TESTS=1.  Their recorded outcome is quoted in the design document.
long_run = pytest.mark.skipif(os.environ.get("FDG_LONG_TESTS", "0") != "1", reason="minutes of oracle time: set FDG_LONG_TESTS=1")


def test_config2_full_size_against_the_oracle(orc):
    net = sy.config(1)                      # 3072 -> 8 x 1024 -> 10, K = 4, 4 workers x 128
    # every tensor within 2e-2 or, eight ReLU layers deep, three times the oracle's own response to a one-ulp change of 0.1 % of the inputs
    rec = run_parity(orc, net, 2 * net.K + 2, grad_tol=2e-2, noise_factor=3.0, loss_tol=1e-2, perturb=False)
    assert not np.isnan(rec[-1]["loss_g"])


@long_run
def test_config2_full_size_all_200_iterations(orc):
    """Configuration 2 as stated (lr 0.05, 200 iterations): loss within 1e-2 of the oracle's at every one of them."""
    net = sy.config(1)
    rec = run_parity(orc, net, net.steps, loss_tol=1e-2, perturb=False)
    assert len(rec) == 200 and not np.isnan(rec[-1]["loss_g"])


@pytest.mark.parametrize("idx,workers,batch", [(3, 8, 8), (4, 16, 2)])
def test_full_width_resnet18_without_relu_every_tensor_of_every_module(orc, idx, workers, batch):
    """Full channel widths (64 .. 512, 32x32 input), K = 4 with 8 workers x 8 samples and K = 8 with 16 workers x 2, lr
    0.05, the networks without their ReLU layers (see tests/test_oracle_pins.py for why): every convolution,
    batch-norm and shortcut gradient of every module within 2e-2 of the oracle (L2 and element by element) at every
    step until the first module has had its second backward pass.  This is where the 256-column CTA-pair kernels, the
    plain and rows-mode weight gradients of the 256- and 512-channel layers, the 4x4-image tiles (eight samples per tile;
    with 2 samples per worker they straddle workers and the batch-norm statistics take their own pass) and the
    stride-2 / 1x1 kernels meet the oracle inside the whole pipeline."""
    net = sy.without_relu(sy.config(idx, n_workers=workers, batch=batch))
    rec = run_parity(orc, net, 2 * net.K + 1, grad_tol=2e-2, elem_tol=3e-2, pair_bn=True, loss_tol=1e-2)
    print(net.name, "worst tensor", max(r.get("grad_err", 0) for r in rec), "worst element", max(r.get("elem_err", 0) for r in rec))


def test_full_width_resnet18_with_relu_loss_and_noise_calibrated_gradients(orc):
    """The benchmark's own network at full width, K = 4, 8 workers x 8 samples: schedule, loss within 1e-2, and every
    tensor within the larger of 2e-2 and three times the oracle's own one-ulp response."""
    net = sy.config(3, n_workers=8, batch=8)
    run_parity(orc, net, 2 * net.K, grad_tol=2e-2, noise_factor=3.0, loss_tol=1e-2)


def test_config3_full_width_diverges_at_lr_0_05_in_the_oracle_too_and_is_stable_at_0_005(orc):
    """The VGG-shaped network (eight convolutions, no normalisation) at full width under the stale gradients: at
    lr 0.05 the ORACLE's loss leaves 1e3 within ten iterations (so a non-finite loss of the library at that step size
    is the method diverging, not a kernel fault); at 0.005, the step size the configuration runs with here, both
    stay finite and the library's loss tracks the oracle's."""
    net = sy.config(2, n_workers=4, batch=8)
    p0 = sy.init_params(net.layers, 0, bf16=True)
    from harness import make_oracle
    o = make_oracle(orc, net, p0)
    worst = 0.0
    for t in range(10):
        lo, _ = o.step(sy.batch_inputs(net, t), sy.batch_labels(net, t), 0.05)
        if not np.isnan(lo):
            worst = max(worst, lo)
    assert worst > 1e3, worst
    assert net.lr == 0.005
    rec = run_parity(orc, net, 12, loss_tol=1e-2, perturb=False)
    assert all(r["loss_g"] < 50.0 for r in rec if not np.isnan(r["loss_g"])) and rec[-1]["loss_g"] < 3.0


@long_run
def test_config3_full_width_50_step_loss_trajectory(orc):
    net = sy.config(2, n_workers=4, batch=8)
    rec = run_parity(orc, net, 50, loss_tol=1e-2, perturb=False)
    assert sum(not np.isnan(r["loss_g"]) for r in rec) == 50 - (net.K - 1)


def _run(net, p0, steps, serial):
    import torch
    from paper_2509_05679_b200 import binding
    # the one-stream run sizes its grids like the concurrent one (a third of the SMs): same contraction splits and
    # batch-norm row chunks, hence the same fp32 summation order
    ctx = make_ctx(net, p0, serial=serial, grid_sms=(torch.cuda.get_device_properties(0).multi_processor_count + 2) // 3 if serial else 0)
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


def test_config5_full_size_schedule_and_invariants():
    """ResNet-18-shaped, K = 8, 16 workers x 256 (M = 4096): the whole stash (about 127 GB, store-all) on one GPU.  Until
    the first module has had its backward pass: the delay schedule on the device equals the closed forms with the maximum
    delay 2(K-1) = 14, everything stays finite, the classifier's bias gradient sums to zero and the weight gradient of
    every convolution in front of a batch-norm is orthogonal to its weights channel by channel."""
    import torch
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 140 * 2**30:
        pytest.skip("needs 140 GB of free device memory")
    net = sy.config(4)
    p0 = sy.init_params(net.layers, 0, bf16=True)
    steps = 2 * net.K - 1
    params, grads, traces = _run(net, p0, steps, serial=False)
    for t, (f, b, v) in enumerate(traces):
        fc, bc, vc = closed_form_trace(net.K, t)
        assert (f == fc).all() and (b == bc).all() and (v == vc).all(), t
    assert traces[-1][1][0] == 0 and traces[-1][2][0] == 0          # module 1 back-propagates batch 0 with weight version 0 at t = 2K-2
    assert np.isfinite(params).all() and np.isfinite(grads).all()
    fc_bias = grads[-net.classes:]
    assert abs(fc_bias.sum()) <= 1e-3 * np.abs(fc_bias).sum()
    off = 0
    shapes = sy.param_shapes(net.layers)
    for idx, (li, name, shape, _) in enumerate(shapes):
        n = int(np.prod(shape))
        if name in ("W", "Wp") and len(shape) == 4 and idx + 1 < len(shapes) and shapes[idx + 1][1].startswith("gamma"):
            w = params[off:off + n].astype(np.float64).reshape(shape[0], -1)
            g = grads[off:off + n].astype(np.float64).reshape(shape[0], -1)
            per_channel = np.abs((w * g).sum(1)) / (np.linalg.norm(w, axis=1) * np.linalg.norm(g, axis=1) + 1e-300)
            assert np.median(per_channel) <= 2e-2, (li, name, float(np.median(per_channel)))
        off += n
    torch.cuda.empty_cache()
