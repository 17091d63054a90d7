"""Pins for the oracle's update rule: stale gradients, worker mixing, reductions (CPU only)."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy


def module_offsets(layers, splits):
    shapes = sy.param_shapes(layers)
    bounds = [0] + list(splits) + [len(layers)]
    offs = [0]
    for k in range(len(bounds) - 1):
        n = sum(int(np.prod(s)) for li, _, s, _ in shapes if bounds[k] <= li < bounds[k + 1])
        offs.append(offs[-1] + n)
    return offs


def data(S, B, in_shape, classes, t):
    g = np.random.default_rng(100 + t)
    return g.standard_normal((S * B,) + in_shape), g.integers(0, classes, S * B).astype(np.int32)


def test_K1_S1_is_ordinary_sgd_backprop(orc):
    """Eq. SGD: W(t+1) = W(t) - eta * (1/B) sum dphi/dW, written out independently in numpy."""
    sizes = [7, 6, 5, 4]
    layers = sy.mlp_layers(sizes)
    B, lr = 5, 0.07
    p = sy.perturb_params(sy.init_params(layers, 3), layers, 4, 0.2).astype(np.float64)
    o = orc.Oracle(layers, [], 1, B, (1, 1, 7), 4)
    o.set_params(p)
    Ws, bs, off = [], [], 0
    for i in range(3):
        n = sizes[i] * sizes[i + 1]
        Ws.append(p[off:off + n].reshape(sizes[i + 1], sizes[i]).copy()); off += n
        bs.append(p[off:off + sizes[i + 1]].copy()); off += sizes[i + 1]
    for t in range(4):
        x, y = data(1, B, (1, 1, 7), 4, t)
        loss_o, _ = o.step(x, y, lr)
        h = [x.reshape(B, 7)]
        for i in range(3):
            z = h[-1] @ Ws[i].T + bs[i]
            h.append(np.maximum(z, 0) if i < 2 else z)
        z = h[-1]
        pz = np.exp(z - z.max(1, keepdims=True)); pz /= pz.sum(1, keepdims=True)
        loss = -np.log(pz[np.arange(B), y]).mean()
        d = pz.copy(); d[np.arange(B), y] -= 1; d /= B
        for i in (2, 1, 0):
            gW, gb = d.T @ h[i], d.sum(0)
            d = (d @ Ws[i]) * (h[i] > 0) if i > 0 else None
            Ws[i] -= lr * gW; bs[i] -= lr * gb
        assert abs(loss - loss_o) < 1e-12
        mine = np.concatenate([np.concatenate([Ws[i].ravel(), bs[i]]) for i in range(3)])
        np.testing.assert_allclose(o.params(), mine, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("net", ["mlp", "resnet"])
def test_stale_gradient_is_plain_backprop_through_the_composite_weights(orc, net):
    """Sec. 3.2/3.3: the gradient module k applies at iteration t is the partial derivative of
    phi(batch tau, W~(tau)) with W~(tau) = col{w_j(tau + j - 1)}, tau = t - 2K + k + 1."""
    if net == "mlp":
        layers = sy.mlp_layers([6, 5, 5, 4, 3]); splits = [2, 4, 6]; in_shape = (1, 1, 6)
    else:
        layers, bs = sy.resnet_layers(widths=(4, 8), blocks=1, in_c=2, classes=3)
        splits = [bs[0], bs[1]]; in_shape = (4, 4, 2)
    K, S, B, lr = len(splits) + 1, 2, 3, 0.05
    offs = module_offsets(layers, splits)
    o = orc.Oracle(layers, splits, S, B, in_shape, 3)
    p0 = sy.perturb_params(sy.init_params(layers, 1), layers, 2, 0.2).astype(np.float64)
    o.set_params(p0)
    hist = [p0.copy()]                 # hist[v] = weights of version v (replicas stay identical)
    batches = []
    checked = 0
    for t in range(3 * K + 2):
        x, y = data(S, B, in_shape, 3, t)
        batches.append((x, y))
        o.step(x, y, lr)
        for s in range(S):
            g = o.grads(s)
            for k in range(1, K + 1):
                tau = t - 2 * K + k + 1
                sl = slice(offs[k - 1], offs[k])
                if tau < 0:
                    assert not g[sl].any()
                    continue
                comp = np.concatenate([hist[tau + j - 1][offs[j - 1]:offs[j]] for j in range(1, K + 1)])
                xb, yb = batches[tau]
                _, ref = orc.plain_loss_grad(layers, 1, B, in_shape, comp, xb[s * B:(s + 1) * B], yb[s * B:(s + 1) * B])
                np.testing.assert_allclose(g[sl], ref[sl], rtol=1e-9, atol=1e-13)
                checked += 1
        hist.append(o.params(0))
        np.testing.assert_array_equal(o.params(0), o.params(1))     # delta(t) = 0 under exact averaging
    assert checked > 2 * K


def test_planted_mistake_current_weights_breaks_the_composite_identity(orc):
    layers = sy.mlp_layers([6, 5, 4, 3]); splits = [2, 4]; K, B = 3, 4
    offs = module_offsets(layers, splits)
    o = orc.Oracle(layers, splits, 1, B, (1, 1, 6), 3)
    o.use_current_weights(True)
    p0 = sy.init_params(layers, 1).astype(np.float64)
    o.set_params(p0)
    hist, batches, bad = [p0.copy()], [], 0
    for t in range(3 * K):
        x, y = data(1, B, (1, 1, 6), 3, t)
        batches.append((x, y))
        o.step(x, y, 0.2)
        g = o.grads(0)
        for k in range(1, K):          # module K has zero delay and cannot show the mistake
            tau = t - 2 * K + k + 1
            if tau < 1:
                continue
            comp = np.concatenate([hist[tau + j - 1][offs[j - 1]:offs[j]] for j in range(1, K + 1)])
            _, ref = orc.plain_loss_grad(layers, 1, B, (1, 1, 6), comp, *batches[tau])
            sl = slice(offs[k - 1], offs[k])
            bad += not np.allclose(g[sl], ref[sl], rtol=1e-9, atol=1e-13)
        hist.append(o.params(0))
    assert bad > 0


def test_worker_average_equals_concatenated_batch_gradient(orc):
    """No batch-norm: mean over S workers of (1/B) sum_{B_s} == (1/(S B)) sum over all samples."""
    layers, _ = sy.vgg_layers(widths=(3, 4), in_c=2, classes=3)
    S, B, in_shape = 4, 2, (4, 4, 2)
    p = sy.perturb_params(sy.init_params(layers, 5), layers, 6, 0.2).astype(np.float64)
    x, y = data(S, B, in_shape, 3, 0)
    per = [orc.plain_loss_grad(layers, 1, B, in_shape, p, x[s * B:(s + 1) * B], y[s * B:(s + 1) * B])[1] for s in range(S)]
    _, whole = orc.plain_loss_grad(layers, 1, S * B, in_shape, p, x, y)       # one worker, batch S*B, c = 1/(S B)
    np.testing.assert_allclose(np.mean(per, 0), whole, rtol=1e-11, atol=1e-14)
    # and the K=1 update with P = 11^T/S moves the weights by exactly lr * that gradient
    o = orc.Oracle(layers, [], S, B, in_shape, 3)
    o.set_params(p)
    o.step(x, y, 0.3)
    np.testing.assert_allclose(o.params(2), p - 0.3 * whole, rtol=1e-11, atol=1e-14)


def ring_P(S, alpha):
    P = np.zeros((S, S))
    for i in range(S):
        for j in ((i - 1) % S, (i + 1) % S):
            P[i, j] = alpha
        P[i, i] = 1 - 2 * alpha
    return P


def test_general_mixing_matrix_form_and_mean_motion(orc):
    """Lemma 2.1 properties of P; W(t+1) = (P (x) I)(W(t) - eta G(t)) (Appendix A); the replica
    mean moves by -(eta/S) sum_s g_s (Appendix B)."""
    S, B, K = 4, 2, 2
    P = ring_P(S, 0.3)
    assert np.allclose(P, P.T) and np.allclose(P.sum(0), 1) and np.allclose(P.sum(1), 1)
    assert max(abs(np.linalg.eigvals(P - np.ones((S, S)) / S))) < 1
    layers = sy.mlp_layers([5, 4, 3]); splits = [2]
    o = orc.Oracle(layers, splits, S, B, (1, 1, 5), 3, P=P, grad_scale=1.0 / (B * S))
    g = np.random.default_rng(9)
    n = o.n_params
    W = g.standard_normal((S, n)) * 0.3            # distinct replicas
    for s in range(S):
        o.set_params(W[s], worker=s)
    eta = 0.1
    for t in range(2 * K + 2):
        x, y = data(S, B, (1, 1, 5), 3, t)
        o.step(x, y, eta)
        G = np.stack([o.grads(s) for s in range(S)])
        Wn = np.stack([o.params(s) for s in range(S)])
        np.testing.assert_allclose(Wn, P @ (W - eta * G), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(Wn.mean(0), W.mean(0) - (eta / S) * G.sum(0), rtol=1e-12, atol=1e-14)
        W = Wn
    assert np.abs(G).max() > 0


def test_complete_graph_alpha_1_over_S_is_exact_averaging(orc):
    S = 3
    P = np.full((S, S), 1.0 / S)                   # Eq. weight_matrix with alpha = 1/S, kappa = S-1
    layers = sy.mlp_layers([5, 4, 3])
    a = orc.Oracle(layers, [2], S, 2, (1, 1, 5), 3, P=P)
    b = orc.Oracle(layers, [2], S, 2, (1, 1, 5), 3)           # default mixing
    p = sy.init_params(layers, 2)
    a.set_params(p); b.set_params(p)
    for t in range(5):
        x, y = data(S, 2, (1, 1, 5), 3, t)
        a.step(x, y, 0.1); b.step(x, y, 0.1)
    np.testing.assert_array_equal(a.params(1), b.params(1))
    np.testing.assert_array_equal(a.params(0), a.params(2))


def test_sgd_closed_form_on_a_hand_made_case(orc):
    """One linear layer, one sample, zero weights: logits 0 => softmax uniform, so
    dW = (1/3 - onehot) x^T and W(1) = -eta dW exactly."""
    layers = [(sy.LINEAR, 2, 3, 1, 1)]
    o = orc.Oracle(layers, [], 1, 1, (1, 1, 2), 3)
    o.set_params(np.zeros(9))
    x = np.array([[2.0, -1.0]]); y = np.array([1], np.int32)
    loss, _ = o.step(x, y, 0.5)
    d = np.array([1 / 3, 1 / 3 - 1, 1 / 3])
    want = np.concatenate([(-0.5 * np.outer(d, x[0])).ravel(), -0.5 * d])
    assert abs(loss - np.log(3)) < 1e-15
    np.testing.assert_allclose(o.params(), want, rtol=1e-14, atol=1e-16)
