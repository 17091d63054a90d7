"""Pins for the oracle's layer arithmetic (CPU only).

Every check compares the oracle with something that is not the oracle: central finite
differences of its own forward pass, torch's autograd on the same tiny network, or a closed form.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from paper_2509_05679_b200 import synth as sy


def tiny_nets():
    mlp = sy.mlp_layers([6, 5, 4, 3])
    vgg, _ = sy.vgg_layers(widths=(3, 4), in_c=2, classes=3)
    res, _ = sy.resnet_layers(widths=(4, 8), blocks=1, in_c=2, classes=3)
    return {"mlp": (mlp, (1, 1, 6), 3), "vgg": (vgg, (4, 4, 2), 3), "resnet": (res, (4, 4, 2), 3)}


def make_case(layers, in_shape, classes, S, B, seed):
    g = np.random.default_rng(seed)
    p = sy.perturb_params(sy.init_params(layers, seed), layers, seed + 1, 0.3).astype(np.float64)
    x = g.standard_normal((S * B,) + in_shape)
    y = g.integers(0, classes, S * B).astype(np.int32)
    return p, x, y


@pytest.mark.parametrize("name", ["mlp", "vgg", "resnet"])
def test_gradient_matches_central_finite_differences(orc, name):
    layers, in_shape, classes = tiny_nets()[name]
    S, B = 2, 3
    p, x, y = make_case(layers, in_shape, classes, S, B, 11)
    # grad_scale 1/(S*B) makes the returned gradient the gradient of the returned mean loss
    loss, grad = orc.plain_loss_grad(layers, S, B, in_shape, p, x, y, grad_scale=1.0 / (S * B))
    g = np.random.default_rng(5)
    idx = g.choice(p.size, size=min(60, p.size), replace=False)
    eps = 1e-5
    worst = 0.0
    for i in idx:
        pp, pm = p.copy(), p.copy()
        pp[i] += eps
        pm[i] -= eps
        lp, _ = orc.plain_loss_grad(layers, S, B, in_shape, pp, x, y, want_grad=False)
        lm, _ = orc.plain_loss_grad(layers, S, B, in_shape, pm, x, y, want_grad=False)
        fd = (lp - lm) / (2 * eps)
        worst = max(worst, abs(fd - grad[i]) / max(abs(fd), abs(grad[i]), 1e-6))
    assert worst <= 1e-4, worst


def torch_forward(layers, params, x, S, B):
    """The same network in torch ops (NCHW), batch-norm statistics per worker."""
    off = 0

    def take(shape):
        nonlocal off
        n = int(np.prod(shape))
        t = params[off:off + n].reshape(shape)
        off += n
        return t

    outs = []
    # parameters are shared by the workers: slice them once, apply per worker
    plan = []
    for kind, cin, cout, stride, flags in layers:
        if kind == sy.LINEAR:
            plan.append(("lin", take((cout, cin)), take((cout,)) if flags & 1 else None))
        elif kind in (sy.CONV3X3, sy.CONV1X1):
            r = 3 if kind == sy.CONV3X3 else 1
            plan.append(("conv", take((cout, r, r, cin)), take((cout,)) if flags & 1 else None, stride, r // 2))
        elif kind == sy.BATCHNORM:
            plan.append(("bn", take((cin,)), take((cin,))))
        elif kind == sy.RES_ADD:
            if flags & 1:
                plan.append(("addp", take((cout, 1, 1, cin)), take((cout,)), take((cout,)), stride))
            else:
                plan.append(("add",))
        else:
            plan.append(({sy.RELU: "relu", sy.MAXPOOL2: "pool", sy.GLOBAL_AVGPOOL: "gap", sy.RES_BEGIN: "begin"}[kind],))
    for s in range(S):
        h = x[s * B:(s + 1) * B].permute(0, 3, 1, 2)
        stack = []
        for op in plan:
            if op[0] == "lin":
                h = h.permute(0, 2, 3, 1).reshape(h.shape[0], -1)
                h = F.linear(h, op[1], op[2])[:, :, None, None]
            elif op[0] == "conv":
                h = F.conv2d(h, op[1].permute(0, 3, 1, 2), op[2], stride=op[3], padding=op[4])
            elif op[0] == "bn":
                h = F.batch_norm(h, None, None, op[1], op[2], training=True, eps=1e-5)
            elif op[0] == "relu":
                h = F.relu(h)
            elif op[0] == "pool":
                h = F.max_pool2d(h, 2)
            elif op[0] == "gap":
                h = h.mean(dim=(2, 3), keepdim=True)
            elif op[0] == "begin":
                stack.append(h)
            elif op[0] == "add":
                h = h + stack.pop()
            elif op[0] == "addp":
                sc = F.conv2d(stack.pop(), op[1].permute(0, 3, 1, 2), None, stride=op[4])
                h = h + F.batch_norm(sc, None, None, op[2], op[3], training=True, eps=1e-5)
        outs.append(h.reshape(h.shape[0], -1))
    return torch.cat(outs, 0)


@pytest.mark.parametrize("name", ["mlp", "vgg", "resnet"])
def test_loss_logits_and_gradient_match_torch_autograd(orc, name):
    layers, in_shape, classes = tiny_nets()[name]
    S, B = 2, 4
    p, x, y = make_case(layers, in_shape, classes, S, B, 23)
    loss, grad = orc.plain_loss_grad(layers, S, B, in_shape, p, x, y, grad_scale=1.0 / (S * B))
    logits = orc.plain_logits(layers, S, B, in_shape, p, x, classes)
    tp = torch.tensor(p, dtype=torch.float64, requires_grad=True)
    tl = torch_forward(layers, tp, torch.tensor(x, dtype=torch.float64), S, B)
    tloss = F.cross_entropy(tl, torch.tensor(y, dtype=torch.long))
    tloss.backward()
    np.testing.assert_allclose(logits, tl.detach().numpy(), rtol=1e-10, atol=1e-12)
    assert abs(loss - tloss.item()) < 1e-12
    np.testing.assert_allclose(grad, tp.grad.numpy(), rtol=1e-8, atol=1e-12)


def test_stride2_conv_and_maxpool_first_max_wins(orc):
    # a stride-2 3x3 conv followed by a pool over a tensor with exact ties
    layers = [(sy.CONV3X3, 1, 2, 2, 1), (sy.MAXPOOL2, 2, 2, 2, 0), (sy.GLOBAL_AVGPOOL, 2, 2, 1, 0), (sy.LINEAR, 2, 2, 1, 1)]
    S, B, in_shape = 1, 2, (8, 8, 1)
    p, x, y = make_case(layers, in_shape, 2, S, B, 3)
    x[:] = 1.0                      # constant image: interior conv outputs tie inside pool windows
    loss, grad = orc.plain_loss_grad(layers, S, B, in_shape, p, x, y, grad_scale=0.5)
    tp = torch.tensor(p, dtype=torch.float64, requires_grad=True)
    tl = torch_forward(layers, tp, torch.tensor(x, dtype=torch.float64), S, B)
    F.cross_entropy(tl, torch.tensor(y, dtype=torch.long)).backward()
    # parameter gradients do not depend on which of the tied maxima receives the gradient
    # only if inputs at the tied positions are equal; here they are (constant image, same taps)
    np.testing.assert_allclose(grad[-6:], tp.grad.numpy()[-6:], rtol=1e-9, atol=1e-12)


def test_softmax_cross_entropy_closed_forms(orc):
    n, c = 5, 10
    y = np.arange(n, dtype=np.int32) % c
    loss, g = orc.softmax_ce(np.full((n, c), 3.25), y, scale=1.0)
    assert abs(loss - np.log(10.0)) < 1e-14                     # uniform logits: ln(classes)
    expect = np.full((n, c), 0.1)
    expect[np.arange(n), y] -= 1.0
    np.testing.assert_allclose(g, expect, atol=1e-15)
    z = np.random.default_rng(0).standard_normal((n, c)) * 4
    l1, g1 = orc.softmax_ce(z, y, 0.25)
    l2, g2 = orc.softmax_ce(z + 1000.0, y, 0.25)                # shift invariance, no overflow
    assert abs(l1 - l2) < 1e-9
    np.testing.assert_allclose(g1, g2, atol=1e-12)
    np.testing.assert_allclose(g1.sum(1), 0.0, atol=1e-15)      # rows of softmax - onehot sum to 0
    # two classes: loss = log(1 + exp(-(z_y - z_other)))
    z2 = np.array([[0.3, -1.1]])
    l, _ = orc.softmax_ce(z2, np.array([0], np.int32), 1.0)
    assert abs(l - np.log1p(np.exp(-1.4))) < 1e-14


def test_bf16_storage_rounding_matches_torch_and_its_properties(orc):
    g = np.random.default_rng(3)
    x = np.concatenate([g.standard_normal(4000) * 10.0 ** g.integers(-6, 6, 4000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 3.3895313892515355e38]])
    got = orc.round_bf16(x)
    want = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(orc.round_bf16(got), got)                 # idempotent
    assert np.all(np.abs(got - x) <= np.abs(x) * 2.0 ** -8)                 # half an ulp of 8 significand bits
    assert orc.round_bf16([1.0 + 2.0 ** -8])[0] == 1.0                      # tie -> even
    assert orc.round_bf16([1.0 + 3 * 2.0 ** -8])[0] == 1.0 + 2.0 ** -6      # tie -> even (up)


def test_bf16_storage_model_stays_close_to_the_fp64_run_and_is_off_by_default(orc):
    layers, bs = sy.resnet_layers(widths=(4, 8), blocks=1, in_c=2, classes=3)
    S, B, in_shape = 2, 3, (4, 4, 2)
    p = sy.round_to_bf16(sy.perturb_params(sy.init_params(layers, 1), layers, 2, 0.2))
    runs = {}
    for mode in (False, True):
        o = orc.Oracle(layers, [bs[0], bs[1]], S, B, in_shape, 3)
        o.storage_bf16(mode)
        o.set_params(p)
        g = np.random.default_rng(0)
        for t in range(7):
            x = sy.round_to_bf16(g.standard_normal((S * B,) + in_shape).astype(np.float32))
            loss, _ = o.step(x, g.integers(0, 3, S * B), 0.05)
        runs[mode] = (loss, o.grads(0))
    assert runs[True][0] != runs[False][0]
    assert abs(runs[True][0] - runs[False][0]) < 2e-2 * runs[False][0]
    d = np.linalg.norm(runs[True][1] - runs[False][1]) / np.linalg.norm(runs[False][1])
    assert 0 < d < 0.1
