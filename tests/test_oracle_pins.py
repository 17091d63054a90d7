"""Pins for the parts of the oracle that the finite-difference and autograd checks leave open (CPU only):
the max-pool tie rule, where the bf16 storage model rounds, and how far a bf16-storage run can be
trusted as a reference for gradients of a deep ReLU network (which fixes the tolerances of the GPU tests).

Expected values are written out by hand or evaluated by straight-line numpy code that shares nothing with
the oracle's layer loops; rounding to bf16 is torch's conversion, not the oracle's.
"""
import numpy as np
import torch

from paper_2509_05679_b200 import synth as sy


def bf16(v):
    """value -> fp32 -> bf16 (round to nearest even), torch's conversions."""
    return torch.tensor(np.asarray(v, dtype=np.float64), dtype=torch.float32).bfloat16().double().numpy()


# ------------------------------------------------------------------------------------------ max-pool ties
TIE_LAYERS = [(sy.CONV1X1, 2, 1, 1, 0), (sy.MAXPOOL2, 1, 1, 2, 0), (sy.GLOBAL_AVGPOOL, 1, 1, 1, 0), (sy.LINEAR, 1, 2, 1, 1)]
# conv W = (1, 1); linear V = (1, -1), b = (0, 0)
TIE_PARAMS = np.array([1.0, 1.0, 1.0, -1.0, 0.0, 0.0])
# sample 0: the four pixels (row-major) are (1,2) (2,1) (0,3) (3,0): the conv output is 3 everywhere, a four-way tie
# sample 1: (0,1) (1,0) (2,3) (1,0): conv output 1, 1, 5, 1, the maximum is the third pixel
TIE_X = np.array([[[[1, 2], [2, 1]], [[0, 3], [3, 0]]], [[[0, 1], [1, 0]], [[2, 3], [1, 0]]]], dtype=np.float64)
TIE_Y = np.array([1, 0], dtype=np.int32)
# By hand (gradient scale 1, i.e. the sum over the two samples): pooled values 3 and 5, logits (3,-3) and (5,-5),
# d loss / d pooled = V . (softmax - onehot) = 2 sigma(6) for sample 0 (label 1) and 2 (sigma(10) - 1) for sample 1
# (label 0).  The conv-weight gradient is that factor times the INPUT PIXEL that won the pool:
#   first maximum wins:  2 sigma(6) (1,2) + 2 (sigma(10)-1) (2,3) = (1.9948731622119211, 3.989837120161247)
#   last maximum wins:   2 sigma(6) (3,0) + ...                   = (5.984982669585383, -0.000272387...)
TIE_DW_FIRST = np.array([1.9948731622119211, 3.989837120161247])
TIE_DW_LAST = np.array([5.984982669585383, -0.00027238721221434226])
TIE_DV = np.array([2.99235514, -2.99235514])
TIE_DB = np.array([0.99748198, -0.99748198])


def test_maxpool_tie_first_maximum_in_row_major_order_receives_the_gradient(orc):
    loss, g = orc.plain_loss_grad(TIE_LAYERS, 1, 2, (2, 2, 2), TIE_PARAMS, TIE_X, TIE_Y, grad_scale=1.0)
    np.testing.assert_allclose(g[:2], TIE_DW_FIRST, rtol=1e-12)
    assert np.abs(g[:2] - TIE_DW_LAST).max() > 1.0            # the other tie rule gives a different conv gradient
    np.testing.assert_allclose(g[2:4], TIE_DV, rtol=1e-7)
    np.testing.assert_allclose(g[4:6], TIE_DB, rtol=1e-7)
    # mean loss: -log softmax_1(3,-3) and -log softmax_0(5,-5)
    assert abs(loss - 0.5 * (np.log1p(np.exp(6.0)) + np.log1p(np.exp(-10.0)))) < 1e-12


# ------------------------------------------------------------------------------------------ bf16 storage points
def storage_case():
    layers = [(sy.CONV1X1, 1, 1, 1, 0), (sy.RES_BEGIN, 1, 1, 1, 0), (sy.CONV1X1, 1, 1, 1, 0), (sy.BATCHNORM, 1, 1, 1, 0),
              (sy.RES_ADD, 1, 1, 1, 0), (sy.LINEAR, 1, 2, 1, 1)]
    # parameters in canonical order: w0, w1, gamma, beta, V[2], b[2]; none of the products below is bf16-exact
    p = np.array([1.2578125, -0.83984375, 1.1, 0.3, 0.7109375, -1.3046875, 0.05, -0.02])
    x = bf16(np.array([0.337, -1.213, 2.031]))
    y = np.array([1, 0, 1], dtype=np.int32)
    return layers, p, x, y


def storage_model_by_hand(p, x, y, round_bn_before_add=False, round_block_conv_gradient=False):
    """The tiny residual block above, straight line, with every storage point of the bf16 model written out."""
    B = len(x)
    w0, w1, gamma, beta, V, b = bf16(p[0]), bf16(p[1]), p[2], p[3], bf16(p[4:6]), p[6:8]     # matrices stored in bf16, vectors not
    h0 = bf16(w0 * x)                                   # conv output: stored
    c = bf16(w1 * h0)                                   # conv output: stored
    mean, var = c.mean(), ((c - c.mean()) ** 2).mean()
    istd = 1.0 / np.sqrt(var + 1e-5)
    xh = (c - mean) * istd
    bn = gamma * xh + beta                              # followed by the add: NOT stored on its own ...
    if round_bn_before_add:
        bn = bf16(bn)
    a = bf16(bn + h0)                                   # ... the sum is rounded once
    z = a[:, None] * V[None, :] + b[None, :]            # logits: fp32 in the library, unrounded here
    e = np.exp(z - z.max(1, keepdims=True))
    sm = e / e.sum(1, keepdims=True)
    onehot = np.eye(2)[y]
    dz = bf16((sm - onehot) / B)                        # stored error gradient
    da = bf16(dz @ V)                                   # the linear layer hands its input gradient on: stored
    s1, s2 = da.sum(), (da * xh).sum()
    gc = bf16(gamma * istd * (da - s1 / B - xh * s2 / B))   # batch-norm hands its input gradient on: stored
    gx = gc * w1                                        # the conv that opens the block hands its gradient to the add unrounded
    if round_block_conv_gradient:
        gx = bf16(gx)
    g = bf16(gx + da)                                   # the add at the block's entry rounds the sum once
    return np.array([(g * x).sum(), (gc * h0).sum(), s2, s1, (dz[:, 0] * a).sum(), (dz[:, 1] * a).sum(), dz[:, 0].sum(), dz[:, 1].sum()])


def test_storage_points_batchnorm_before_add_and_block_opening_conv_gradient_are_not_rounded(orc):
    layers, p, x, y = storage_case()
    o = orc.Oracle(layers, [], 1, 3, (1, 1, 1), 2)
    o.storage_bf16(True)
    o.set_params(p)
    o.step(x.reshape(3, 1, 1, 1), y, 0.0)
    g = o.grads(0)
    want = storage_model_by_hand(p, x, y)
    np.testing.assert_allclose(g, want, rtol=1e-10, atol=1e-14)
    # the two placements the oracle does NOT use give measurably different gradients on this case,
    # so the comparison above does pin them
    for alt in (dict(round_bn_before_add=True), dict(round_block_conv_gradient=True)):
        other = storage_model_by_hand(p, x, y, **alt)
        assert np.abs(other - want).max() > 1e-4 * np.abs(want).max(), alt
    # and with the storage model off the same network gives the unrounded result
    o2 = orc.Oracle(layers, [], 1, 3, (1, 1, 1), 2)
    o2.set_params(p)
    o2.step(x.reshape(3, 1, 1, 1), y, 0.0)
    assert np.abs(o2.grads(0) - want).max() > 1e-4 * np.abs(want).max()


# ------------------------------------------------------------------------------------------ what a bf16 run can be held to
def _oracle_gradient(orc, net, x, y):
    p0 = sy.round_to_bf16(sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1))
    o = orc.Oracle(net.layers, [], net.n_workers, net.batch, (net.in_h, net.in_w, net.in_c), net.classes)
    o.storage_bf16(True)
    o.set_params(p0)
    o.step(x, y, 0.0)
    return np.mean([o.grads(s) for s in range(net.n_workers)], axis=0)


def test_one_ulp_on_a_thousandth_of_the_inputs_moves_deep_relu_gradients_by_tens_of_percent_but_not_relu_free_ones(orc):
    """Why the GPU tests hold every tensor of a DEEP network to 2e-2 only on ReLU-free networks.

    With bf16 storage every stored tensor re-draws its rounding, so two evaluations that differ anywhere (the
    library accumulates in fp32, the oracle in fp64) differ by about one rounding (2^-9 relative) in every stored
    tensor a few layers later.  A ReLU whose input moves by a relative eps flips the mask of about eps of its
    elements, and each flip changes a gradient term by its full size: the gradient moves by about sqrt(eps) per ReLU
    layer, 5-8 % for eps = 2^-9 .. 2^-8, and the layers add up.  Measured here on the ORACLE ALONE: moving 0.1 % of the
    input values by one bf16 ulp changes the gradients of the ResNet-18-shaped network (width / 4, 2 x 4 samples) by
    20-35 % in every convolution below the last block, while the same network without its ReLU layers moves by about
    1 % in every tensor.  So no implementation can be held to 2e-2 against this oracle on the first, and every one can
    on the second.  (gamma and beta of a batch-norm are compared as one tensor there, see harness.gradient_groups.)"""
    from harness import grad_rel_l2, ulp_perturbed
    net = sy.config(3, n_workers=2, batch=4, width_div=4)
    net.splits = []
    x, y = sy.batch_inputs(net, 0), sy.batch_labels(net, 0)
    xp = ulp_perturbed(x, 1e-3, 5)
    assert 0 < np.count_nonzero(xp != x) <= 1e-3 * x.size + 1
    _, _, with_relu = grad_rel_l2(_oracle_gradient(orc, net, xp, y), _oracle_gradient(orc, net, x, y), net.layers)
    convs = [v for k, v in with_relu.items() if k.endswith(".W") and not k.startswith("L68")]
    print("with ReLU   : conv tensors min / median / max", min(convs), float(np.median(convs)), max(convs))
    assert np.median(convs) > 0.10 and min(convs[:8]) > 0.10
    lin = sy.without_relu(net)
    worst, where, _ = grad_rel_l2(_oracle_gradient(orc, lin, xp, y), _oracle_gradient(orc, lin, x, y), lin.layers, pair_bn=True)
    print("without ReLU: worst tensor", worst, where)
    assert worst < 1.5e-2


def test_relu_free_network_shows_a_wrong_weight_version_at_the_gpu_tests_tolerance(orc):
    """The ReLU-free ResNet-18-shaped run of the GPU tests (lr 0.05, every tensor within 2e-2 at every step) would
    catch a backward pass that reads the wrong weight version: planted in the oracle (current weights instead of
    the stashed ones, Sec. 3.2), the first module's tensors are off by more than 5e-2 two steps after its first
    update, while the run itself stays stable (loss below 4)."""
    from harness import grad_rel_l2
    net = sy.without_relu(sy.config(3, n_workers=2, batch=4, width_div=4))
    p0 = sy.round_to_bf16(sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1))
    runs = []
    for planted in (False, True):
        o = orc.Oracle(net.layers, net.splits, net.n_workers, net.batch, (net.in_h, net.in_w, net.in_c), net.classes)
        o.storage_bf16(True)
        o.set_params(p0)
        o.use_current_weights(planted)
        runs.append(o)
    for t in range(2 * net.K + 1):
        x, y = sy.batch_inputs(net, t), sy.batch_labels(net, t)
        losses = [o.step(x, y, net.lr)[0] for o in runs]
        assert np.isnan(losses[0]) or losses[0] < 4.0
    ga, gb = (np.mean([o.grads(s) for s in range(net.n_workers)], axis=0) for o in runs)
    _, _, per = grad_rel_l2(gb, ga, net.layers, pair_bn=True)
    first_module = [v for k, v in per.items() if int(k[1:].split(".")[0]) < net.splits[0]]
    assert min(first_module) > 5e-2, per
