"""fdg_options.grid_sms: the SM count the persistent kernels (tensor-core convolutions, streamed batch-norm) size their
grids, contraction splits and row chunks for, so that kernels of different module streams (the concurrency of Sec. 3.2)
run side by side.  It must change nothing but fp32 summation order."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import make_ctx, grad_rel_l2

pytestmark = pytest.mark.gpu


def _net():
    # ReLU-free, so that a different summation order cannot flip a mask (see tests/test_oracle_pins.py)
    layers, bs = sy.resnet_layers(widths=(64, 128), blocks=1, in_c=3, classes=10)
    return sy.without_relu(sy.Net("resnet-64-128", layers, [bs[0], bs[1]], 32, 32, 3, 10, 2, 4, 0.05, "bf16"))


def _run(net, p0, steps, **kw):
    import torch
    from paper_2509_05679_b200 import binding
    ctx = make_ctx(net, p0, **kw)
    sms = ctx.grid_sms
    for t in range(steps):
        ctx.step(binding.to_device(net.dtype, sy.batch_inputs(net, t)), torch.from_numpy(sy.batch_labels(net, t)).cuda())
    out = ctx.params(), ctx.grads(), ctx.trace()
    ctx.close()
    return sms, out


def test_automatic_choice_and_clamping():
    import torch
    device_sms = torch.cuda.get_device_properties(0).multi_processor_count
    net = _net()
    p0 = sy.round_to_bf16(sy.init_params(net.layers, 0))
    # module streams: a third of the device; one stream: nothing runs beside a kernel, all of it; explicit values are clamped
    for kw, want in ((dict(), (device_sms + 2) // 3), (dict(serial=True), device_sms), (dict(grid_sms=17), 17), (dict(grid_sms=10 ** 6), device_sms)):
        ctx = make_ctx(net, p0, **kw)
        assert ctx.grid_sms == want, (kw, ctx.grid_sms)
        ctx.close()


def test_grid_size_changes_only_the_summation_order():
    import torch
    device_sms = torch.cuda.get_device_properties(0).multi_processor_count
    net = _net()
    p0 = sy.round_to_bf16(sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1))
    steps = 2 * net.K + 1
    runs = {}
    for sms in (0, device_sms, 16, 5):
        got, runs[sms] = _run(net, p0, steps, grid_sms=sms)
        assert got == (sms or (device_sms + 2) // 3)
    ref_p, ref_g, ref_t = runs[0]
    for sms, (p, g, tr) in runs.items():
        assert all((a == b).all() for a, b in zip(tr, ref_t))                # the schedule does not depend on it
        worst, where, _ = grad_rel_l2(g, ref_g, net.layers, pair_bn=True)
        assert worst < 1e-2, (sms, worst, where)                             # bf16 storage re-rounds what a different order moved
        assert np.abs(p - ref_p).max() <= 1e-3 * np.abs(ref_p).max(), sms
    # the same size twice: bit-identical, whatever the streams
    _, again = _run(net, p0, steps, grid_sms=16)
    assert np.array_equal(again[0], runs[16][0]) and np.array_equal(again[1], runs[16][1])
    _, one_stream = _run(net, p0, steps, grid_sms=16, serial=True)
    assert np.array_equal(one_stream[0], runs[16][0])
