"""Pins for the delay schedule that the oracle's message passing produces (CPU only)."""
import os

import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "schedule_K3.txt")


def chain_net(K):
    """K tiny linear modules (one linear layer + relu each, last one bare)."""
    sizes = [4] + [3] * (K - 1) + [3]
    layers = sy.mlp_layers(sizes)
    splits = [2 * k for k in range(1, K)]
    return layers, splits


def run_trace(orc, K, T, S=1, B=2):
    layers, splits = chain_net(K)
    o = orc.Oracle(layers, splits, S, B, (1, 1, 4), 3)
    o.set_params(sy.init_params(layers, 0))
    g = np.random.default_rng(0)
    rows = []
    for t in range(T):
        o.step(g.standard_normal((S * B, 4)), g.integers(0, 3, S * B), 0.01)
        f, b, v, m = o.trace()
        for k in range(K):
            rows.append((t, k + 1, int(f[k]), int(b[k]), int(v[k])))
    return rows, o.trace()[3]


def token_recount(K, T):
    """Brute force: push batch ids through K boxes, one hop per iteration, and back again."""
    act_box = [None] * K      # what box k will forward in this iteration
    grad_box = [None] * K     # what box k will back-propagate in this iteration
    fwd_version = [dict() for _ in range(K)]
    rows = []
    for t in range(T):
        act_box[0] = t
        nxt_act, nxt_grad = [None] * K, [None] * K
        for k in range(K):
            f = act_box[k]
            b = None
            if f is not None:
                fwd_version[k][f] = t
                if k + 1 < K:
                    nxt_act[k + 1] = f
                else:
                    b = f
            if k + 1 < K and grad_box[k] is not None:
                b = grad_box[k]
            if b is not None and k > 0:
                nxt_grad[k - 1] = b
            rows.append((t, k + 1, -1 if f is None else f, -1 if b is None else b,
                         -1 if b is None else fwd_version[k][b]))
        act_box, grad_box = nxt_act, nxt_grad
    return rows


def test_trace_matches_hand_written_table_for_three_modules(orc):
    want = [tuple(int(v) for v in ln.split()) for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    got, _ = run_trace(orc, 3, 9)
    assert got == want


@pytest.mark.parametrize("K", range(1, 9))
def test_trace_matches_closed_forms_and_token_recount(orc, K):
    T = 4 * K + 1
    got, max_stash = run_trace(orc, K, T)
    assert got == token_recount(K, T)
    for (t, k, f, b, v) in got:
        tf, tb, ver = t - k + 1, t - 2 * K + k + 1, t - 2 * K + 2 * k
        assert f == (tf if tf >= 0 else -1)
        assert b == (tb if tb >= 0 else -1)
        assert v == (ver if tb >= 0 else -1)
        if tb >= 0:
            assert ver == tb + k - 1          # the version the forward pass of that batch used
    # Appendix A: gradients used at iteration t are those of batches t-2K+2 (k=1) ... t-K+1 (k=K)
    last = [r for r in got if r[0] == T - 1]
    assert [r[3] for r in last] == [T - 1 - 2 * K + 1 + k for k in range(1, K + 1)]
    # a batch stays in module k's stash for 2(K-k) iterations
    assert list(max_stash) == [2 * (K - k) + 1 for k in range(1, K + 1)]


def test_first_update_of_module_k_happens_at_2K_minus_k_minus_1(orc):
    K = 4
    layers = sy.mlp_layers([4, 8, 8, 8, 3])
    splits = [2, 4, 6]
    o = orc.Oracle(layers, splits, 1, 2, (1, 1, 4), 3)
    p0 = sy.init_params(layers, 0).astype(np.float64)
    o.set_params(p0)
    g = np.random.default_rng(1)
    first_change = {}
    # module boundaries in the parameter vector
    sizes = [4 * 8 + 8, 8 * 8 + 8, 8 * 8 + 8, 8 * 3 + 3]
    offs = np.cumsum([0] + sizes)
    for t in range(10):
        o.step(g.standard_normal((2, 4)) + 1.0, g.integers(0, 3, 2), 0.1)
        p = o.params()
        for k in range(K):
            if k not in first_change and np.any(p[offs[k]:offs[k + 1]] != p0[offs[k]:offs[k + 1]]):
                first_change[k] = t
    assert first_change == {k: 2 * K - (k + 1) - 1 for k in range(K)}
