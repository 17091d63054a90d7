"""General mixing matrix P on the GPU (paper Sec. 2.3 Eq. weight_matrix, Sec. 3.3 Eq. dl_update (a)/(b), Sec. 5 Eq.
max_consensus_error): one weight replica per worker, each worker's own stale gradient, w_s(t+1) = sum_r P_sr (w_r - lr g_r).
fp32 path against the oracle's general-P path: every worker's parameters within 1e-5 after every step, the delay
schedule bit-exact, the consensus error delta(t) against its definition evaluated on the oracle's replicas."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import closed_form_trace, max_rel_err

pytestmark = pytest.mark.gpu


def weight_matrix(edges, S, alpha):
    """Eq. weight_matrix: P_ij = alpha on edges, 1 - kappa_i alpha on the diagonal, 0 elsewhere."""
    P = np.zeros((S, S))
    for i, j in edges:
        P[i, j] = P[j, i] = alpha
    kappa = (P > 0).sum(1)
    assert alpha < 1.0 / kappa.max()                     # the admissible range of alpha
    P[np.arange(S), np.arange(S)] = 1.0 - kappa * alpha
    return P


def graphs(S):
    return {"ring": [(i, (i + 1) % S) for i in range(S)], "line": [(i, i + 1) for i in range(S - 1)],
            "complete": [(i, j) for i in range(S) for j in range(i + 1, S)]}


def consensus_error(params_per_worker, layers):
    """delta = max over layers and workers of || w_{s,l} - mean_s w_{s,l} ||_2, straight from the definition."""
    W = np.asarray(params_per_worker, dtype=np.float64)
    mean = W.mean(0)
    worst, off, by_layer = 0.0, 0, {}
    for li, name, shape, _ in sy.param_shapes(layers):
        n = int(np.prod(shape))
        by_layer.setdefault(li, []).append(slice(off, off + n))
        off += n
    for sls in by_layer.values():
        idx = np.r_[tuple(sls)]
        worst = max(worst, max(np.linalg.norm(W[s, idx] - mean[idx]) for s in range(W.shape[0])))
    return worst


def nets():
    mlp = sy.Net("mlp-mix", sy.mlp_layers([24, 32, 16, 10]), [2], 1, 1, 24, 10, 4, 6, 0.1, "fp32")
    layers, bs = sy.resnet_layers(widths=(8, 16), blocks=1, in_c=3, classes=10)
    res = sy.without_relu(sy.Net("resnet-mix", layers, [bs[0], bs[1]], 8, 8, 3, 10, 4, 3, 0.05, "fp32"))
    ragged = sy.Net("mlp-ragged-mix", sy.mlp_layers([22, 33, 17, 10]), [2], 1, 1, 22, 10, 4, 3, 0.1, "fp32")     # windows off 16-byte boundaries
    return {"mlp": mlp, "resnet": res, "ragged": ragged}


def run_pair(orc, net, P, steps, distinct, lr=None):
    import torch
    from paper_2509_05679_b200 import binding
    lr = net.lr if lr is None else lr
    S = net.n_workers
    p0 = sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1)
    reps = [p0 + (0.02 * np.random.default_rng(100 + s).standard_normal(p0.size)).astype(np.float32) if distinct else p0 for s in range(S)]
    o = orc.Oracle(net.layers, net.splits, S, net.batch, (net.in_h, net.in_w, net.in_c), net.classes, P=P)
    ctx = binding.Context(net.layers, net.splits, S, net.batch, lr, dtype="fp32", in_shape=(net.in_h, net.in_w, net.in_c),
                          num_classes=net.classes, mixing=P)
    ctx.set_params(p0)
    for s in range(S):
        o.set_params(reps[s], worker=s)
        if distinct:
            ctx.set_params_worker(s, reps[s])
    deltas = [ctx.consensus_error()]
    assert abs(deltas[0] - consensus_error(reps, net.layers)) <= 1e-6 * max(1.0, deltas[0])
    for t in range(steps):
        x, y = sy.batch_inputs(net, t), sy.batch_labels(net, t)
        lo, _ = o.step(x, y, lr)
        lg = ctx.step(binding.to_device("fp32", x), torch.from_numpy(y).cuda(), want_loss=True)
        fo, bo, vo, _ = o.trace()
        fg, bg, vg = ctx.trace()
        fc, bc, vc = closed_form_trace(net.K, t)
        assert (fg == fo).all() and (bg == bo).all() and (vg == vo).all() and (fg == fc).all() and (bg == bc).all() and (vg == vc).all()
        assert (np.isnan(lo) and np.isnan(lg)) or abs(lg - lo) <= 1e-5 * abs(lo)
        for s in range(S):
            err, where = max_rel_err(ctx.params_worker(s), o.params(s), net.layers)
            assert err <= 1e-5, (t, s, err, where)
            go, gg = o.grads(s), ctx.grads_worker(s)
            assert np.abs(gg - go).max() <= 1e-5 * max(np.abs(go).max(), 1e-30) + 1e-9, (t, s)
        d = ctx.consensus_error()
        want = consensus_error([o.params(s) for s in range(S)], net.layers)
        assert abs(d - want) <= 1e-5 * want + 2e-5, (t, d, want)       # the replicas themselves carry fp32 rounding of about 1e-6 of their norm
        deltas.append(d)
    ctx.close()
    return deltas


@pytest.mark.parametrize("graph,alpha", [("ring", 0.3), ("line", 0.4)])
@pytest.mark.parametrize("name", ["mlp", "resnet", "ragged"])
def test_general_mixing_matrix_matches_the_oracle_for_every_worker(orc, name, graph, alpha):
    net = nets()[name]
    P = weight_matrix(graphs(net.n_workers)[graph], net.n_workers, alpha)
    deltas = run_pair(orc, net, P, 2 * net.K + 3, distinct=True)
    assert deltas[0] > 0 and all(np.isfinite(deltas))


def test_without_gradient_steps_the_consensus_error_contracts_by_the_spectral_radius(orc):
    """lr = 0: W(t+1) = (P (x) I) W(t).  The deviation from the mean obeys D(t+1) = (P - 11^T/S) D(t), whose norm summed over
    the workers contracts by gamma = rho(P - 11^T/S) < 1 per step (Lemma 2.1); the maximum over workers is within sqrt(S)
    of that sum, hence delta(t) <= sqrt(S) gamma^t delta(0)."""
    net = nets()["mlp"]
    S = net.n_workers
    P = weight_matrix(graphs(S)["ring"], S, 0.3)
    gamma = np.abs(np.linalg.eigvalsh(P - np.ones((S, S)) / S)).max()
    assert gamma < 1
    deltas = run_pair(orc, net, P, 8, distinct=True, lr=0.0)
    for t, d in enumerate(deltas):
        assert d <= np.sqrt(S) * gamma ** t * deltas[0] * (1 + 1e-4) + 1e-7, (t, d, deltas[0], gamma)
    assert deltas[-1] < 0.2 * deltas[0]


def test_complete_graph_with_alpha_one_over_S_equals_the_single_copy_path(orc):
    """P = (1/S) 1 1^T given explicitly (S replicas, per-worker gradients, mixing kernel) against the default path (one
    copy, average inside the weight-gradient contraction): same weights up to fp32 summation order, delta(t) = 0."""
    import torch
    from paper_2509_05679_b200 import binding
    net = nets()["resnet"]
    S = net.n_workers
    P = np.full((S, S), 1.0 / S)                  # complete graph, alpha = 1/S < 1/(S-1): the exact average
    p0 = sy.perturb_params(sy.init_params(net.layers, 0), net.layers, 7, 0.1)
    kw = dict(dtype="fp32", in_shape=(net.in_h, net.in_w, net.in_c), num_classes=net.classes)
    a = binding.Context(net.layers, net.splits, S, net.batch, net.lr, mixing=P, **kw)
    b = binding.Context(net.layers, net.splits, S, net.batch, net.lr, kernel_path=1, **kw)
    a.set_params(p0)
    b.set_params(p0)
    for t in range(2 * net.K + 2):
        x, y = binding.to_device("fp32", sy.batch_inputs(net, t)), torch.from_numpy(sy.batch_labels(net, t)).cuda()
        a.step(x, y)
        b.step(x, y)
        pb = b.params()
        for s in range(S):
            err, where = max_rel_err(a.params_worker(s), pb, net.layers)
            assert err <= 1e-5, (t, s, err, where)
        assert a.consensus_error() <= 1e-5
        ga, gb = a.grads(), b.grads()
        assert np.abs(ga - gb).max() <= 1e-5 * max(np.abs(gb).max(), 1e-30) + 1e-9
    a.close()
    b.close()


def test_mixing_matrix_argument_checks():
    from paper_2509_05679_b200 import binding
    net = nets()["mlp"]
    bad = np.full((4, 4), 0.3)
    with pytest.raises(binding.FdgError) as e:
        binding.Context(net.layers, net.splits, 4, net.batch, net.lr, dtype="fp32", in_shape=(1, 1, 24), num_classes=10, mixing=bad)
    assert e.value.status == 1
    ctx = binding.Context(net.layers, net.splits, 4, net.batch, net.lr, dtype="fp32", in_shape=(1, 1, 24), num_classes=10)
    ctx.set_params(sy.init_params(net.layers, 0))
    with pytest.raises(binding.FdgError):
        ctx.set_params_worker(1, sy.init_params(net.layers, 0))          # no replicas without a mixing matrix
    assert ctx.consensus_error() == 0.0
    ctx.close()
