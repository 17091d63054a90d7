"""bf16 path (bf16 activations / weight copies / error gradients, fp32 accumulation, fp32 master
weights) against the fp64 oracle: bit-exact schedule, gradients within 2e-2 (per tensor, relative
L2), loss trajectory within 1e-2 (relative, every step, 50 steps)."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import run_parity

pytestmark = pytest.mark.gpu
GRAD_TOL, LOSS_TOL = 2e-2, 1e-2


def test_config2_shaped_mlp_50_step_loss_trajectory(orc):
    net = sy.config(1, n_workers=4, batch=32, width_div=4)
    rec = run_parity(orc, net, 50, grad_tol=GRAD_TOL, loss_tol=LOSS_TOL, perturb=False)
    assert sum(not np.isnan(r["loss_g"]) for r in rec) == 50 - (net.K - 1)


def test_config3_shaped_vgg(orc):
    net = sy.config(2, n_workers=2, batch=4, width_div=4)
    run_parity(orc, net, 3 * net.K, grad_tol=GRAD_TOL, loss_tol=LOSS_TOL)


def test_config4_shaped_resnet(orc):
    net = sy.config(3, n_workers=2, batch=4, width_div=4)
    run_parity(orc, net, 3 * net.K, grad_tol=GRAD_TOL, loss_tol=LOSS_TOL)


def test_config5_shaped_resnet_eight_modules(orc):
    net = sy.config(4, n_workers=2, batch=2, width_div=8)
    run_parity(orc, net, 2 * net.K + 2, grad_tol=GRAD_TOL, loss_tol=LOSS_TOL)
