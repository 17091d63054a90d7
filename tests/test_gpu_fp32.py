"""fp32 path of the library against the oracle: bit-exact schedule, parameters within max
relative error 1e-5 after every step (per tensor, |a-b| / max(|b|, 0.1 rms(b)))."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import run_parity, make_ctx

pytestmark = pytest.mark.gpu
TOL = 1e-5


def as_fp32(net):
    net.dtype = "fp32"
    return net


def test_config1_mlp_20_iterations(orc):
    net = sy.config(0)
    rec = run_parity(orc, net, net.steps, param_tol=TOL, loss_tol=1e-5, perturb=False, kink_guard=2e-6)
    assert len(rec) == 20 and not np.isnan(rec[-1]["loss_g"])


def test_mlp_four_modules_ragged_sizes(orc):
    net = sy.Net("mlp-k4", sy.mlp_layers([70, 33, 65, 17, 5]), [2, 4, 6], 1, 1, 70, 5, 3, 7, 0.05, "fp32")
    run_parity(orc, net, 4 * net.K + 2, param_tol=TOL, loss_tol=1e-5)


def test_vgg_shaped_four_modules(orc):
    layers, starts = sy.vgg_layers(widths=(6, 10, 12, 20), in_c=3, classes=10)
    net = sy.Net("vgg-small", layers, starts[1:], 16, 16, 3, 10, 2, 3, 0.05, "fp32")
    run_parity(orc, net, 4 * net.K, param_tol=TOL, loss_tol=1e-5, grad_tol=0.2, grad_best_tol=1e-5)


def test_resnet_shaped_four_modules_per_worker_batchnorm(orc):
    net = as_fp32(sy.config(3, n_workers=2, batch=3, width_div=8))
    rec = run_parity(orc, net, 4 * net.K, param_tol=TOL, loss_tol=1e-5, grad_tol=0.2, grad_best_tol=1e-5)
    assert rec[-1]["grad_err"] > 0


def test_resnet_shaped_eight_modules_max_delay(orc):
    net = as_fp32(sy.config(4, n_workers=2, batch=2, width_div=16))
    run_parity(orc, net, 2 * net.K + 3, param_tol=TOL, loss_tol=1e-5)


def test_single_module_single_worker_is_plain_sgd(orc):
    net = as_fp32(sy.config(3, n_workers=1, batch=4, width_div=8, K=1))
    run_parity(orc, net, 3, param_tol=TOL, loss_tol=1e-5)


def test_serial_and_concurrent_modes_are_bit_identical():
    import torch
    from paper_2509_05679_b200 import binding
    net = as_fp32(sy.config(3, n_workers=2, batch=4, width_div=8))
    p0 = sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1)
    outs, sms = [], 0
    for serial in (False, True):
        ctx = make_ctx(net, p0, serial=serial, grid_sms=sms)
        sms = ctx.grid_sms                 # the one-stream run sizes its grids like the concurrent one: same summation order
        for t in range(3 * net.K):
            x, y = binding.to_device("fp32", sy.batch_inputs(net, t)), torch.from_numpy(sy.batch_labels(net, t)).cuda()
            ctx.step(x, y)                 # asynchronous: steps of different modules overlap
            ctx.wait_ingest()              # x and y may be released once the library has copied them
        outs.append(ctx.params())
        ctx.close()
    assert np.array_equal(outs[0], outs[1])


def test_host_buffer_entry_point_matches_device_entry_point():
    import torch
    from paper_2509_05679_b200 import binding
    net = sy.config(0)
    p0 = sy.init_params(net.layers, 0)
    a, b = make_ctx(net, p0), make_ctx(net, p0)
    for t in range(5):
        x, y = sy.batch_inputs(net, t), sy.batch_labels(net, t)
        la = a.step(binding.to_device("fp32", x), torch.from_numpy(y).cuda(), want_loss=True)
        lb = b.step_host(x, y, want_loss=True)
        assert la == lb or (np.isnan(la) and np.isnan(lb))
    assert np.array_equal(a.params(), b.params())
    a.close(); b.close()


def test_error_paths_do_not_touch_the_gpu_state():
    from paper_2509_05679_b200 import binding
    layers, bs = sy.resnet_layers(widths=(8, 16), blocks=1, in_c=3, classes=10)
    with pytest.raises(binding.FdgError) as e:
        binding.Context(layers, [bs[0] + 2], 1, 2, 0.1, dtype="fp32", in_shape=(8, 8, 3))      # cuts a residual block
    assert e.value.status == 2
    with pytest.raises(binding.FdgError) as e:
        binding.Context(layers, [5, 5], 1, 2, 0.1, dtype="fp32", in_shape=(8, 8, 3))           # not increasing
    assert e.value.status == 2
    with pytest.raises(binding.FdgError) as e:
        binding.Context(sy.mlp_layers([8, 4, 3]), [], 1, 2, 0.1, dtype="fp32", in_shape=(1, 1, 9), num_classes=3)
    assert e.value.status == 3
    ctx = binding.Context(sy.mlp_layers([8, 4, 3]), [], 1, 2, 0.1, dtype="fp32", in_shape=(1, 1, 8), num_classes=3)
    with pytest.raises(binding.FdgError) as e:
        ctx.step(1, 1)                                                                          # no parameters yet
    assert e.value.status == 8
    ctx.close()


def test_maxpool_tie_goes_to_the_first_maximum_as_in_the_oracle():
    """The hand-computed four-way tie of tests/test_oracle_pins.py through the library: the conv-weight gradient
    depends on which tied pixel receives the pooled gradient."""
    import torch
    from paper_2509_05679_b200 import binding
    from test_oracle_pins import TIE_LAYERS, TIE_PARAMS, TIE_X, TIE_Y, TIE_DW_FIRST, TIE_DV, TIE_DB
    net = sy.Net("tie", TIE_LAYERS, [], 2, 2, 2, 2, 1, 2, 0.0, "fp32")
    ctx = make_ctx(net, TIE_PARAMS.astype(np.float32))
    ctx.step(binding.to_device("fp32", TIE_X.astype(np.float32)), torch.from_numpy(TIE_Y).cuda(), want_loss=True)
    g = ctx.grads().astype(np.float64) * 2.0          # the library averages over the two samples
    ctx.close()
    np.testing.assert_allclose(g[:2], TIE_DW_FIRST, rtol=1e-5)
    np.testing.assert_allclose(g[2:4], TIE_DV, rtol=1e-5)
    np.testing.assert_allclose(g[4:6], TIE_DB, rtol=1e-5)


def test_param_layout_matches_the_canonical_order_and_addresses_single_tensors():
    """fdg_param_layout against the layer list: names, shapes, contiguous offsets, module ownership; a value planted
    through one record's offset comes back from fdg_params at that tensor and nowhere else."""
    net = sy.config(3, n_workers=2, batch=2, width_div=8)
    p0 = sy.init_params(net.layers, 0)
    ctx = make_ctx(as_fp32(net), p0)
    lay = ctx.param_layout()
    want = sy.param_shapes(net.layers)
    assert [(l, r, s) for l, _, r, s, _, _ in lay] == [(li, name, tuple(shape)) for li, name, shape, _ in want]
    off = 0
    bounds = [0] + list(net.splits) + [len(net.layers)]
    for layer, module, role, shape, offset, count in lay:
        assert offset == off and count == int(np.prod(shape))
        assert bounds[module] <= layer < bounds[module + 1]
        off += count
    assert off == ctx.n_params == p0.size
    layer, module, role, shape, offset, count = lay[len(lay) // 2]
    p1 = p0.copy()
    p1[offset:offset + count] = 0.5
    ctx.set_params(p1)
    back = ctx.params()
    assert np.all(back[offset:offset + count] == 0.5) and np.array_equal(np.delete(back, np.s_[offset:offset + count]), np.delete(p0, np.s_[offset:offset + count]))
    ctx.close()


def test_join_orders_a_caller_stream_behind_the_steps():
    """fdg_join: work the caller enqueues on its own stream afterwards runs after the last update.  An event recorded
    behind the join must complete no earlier than an event the library's last kernel precedes: after synchronising the
    caller's stream alone, the device holds the final weights (a second read after a full device sync is identical)."""
    import torch
    from paper_2509_05679_b200 import binding
    net = as_fp32(sy.config(3, n_workers=2, batch=4, width_div=8))
    ctx = make_ctx(net, sy.init_params(net.layers, 0))
    xs = [binding.to_device("fp32", sy.batch_inputs(net, t)) for t in range(3)]
    ys = [torch.from_numpy(sy.batch_labels(net, t)).cuda() for t in range(3)]
    mine = torch.cuda.Stream()
    for t in range(2 * net.K + 1):
        ctx.step(xs[t % 3], ys[t % 3])
    ctx.join(mine.cuda_stream)
    done = torch.cuda.Event()
    done.record(mine)
    done.synchronize()
    first = ctx.params()
    torch.cuda.synchronize()
    assert np.array_equal(first, ctx.params())
    ctx.close()
