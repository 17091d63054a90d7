"""Worker groups: a module may run its layers once per group of workers (so that a group's tensors stay in
L2 between kernels) and add the groups' parameter gradients.  Nothing in the method changes: the rows of
a batch are independent except inside one worker's batch-norm statistics and inside the sums over all
rows that form the averaged gradient, and a group always holds whole workers.  So a grouped run must pass
the same parity checks against the oracle, and must agree with the ungrouped run up to fp32 summation order."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy
from harness import run_parity, make_ctx

pytestmark = pytest.mark.gpu


def _tensor_core_net():
    """Channel counts in multiples of 64 (the tensor-core kernels' eligibility), two modules: stem, an identity
    block and a stride-2 projection block in the first (the grouped one), an identity block and the head in the second."""
    layers, bs = sy.resnet_layers(widths=(64, 128), blocks=2, in_c=3, classes=10)
    # blocks: 64 id, 64 id, 128 proj, 128 id  ->  module 1 = stem + blocks 0..2, module 2 = block 3 + head
    return sy.Net("resnet-64-128", layers, [bs[3]], 8, 8, 3, 10, 4, 16, 0.02, "bf16")


def test_fp32_resnet_grouped_matches_oracle(orc):
    net = sy.config(3, n_workers=4, batch=3, width_div=8)
    net.dtype = "fp32"
    run_parity(orc, net, 3 * net.K, param_tol=1e-5, loss_tol=1e-5, grad_tol=0.2, grad_best_tol=1e-5, worker_groups=2)


def test_fp32_ragged_mlp_grouped_windows_that_start_off_a_16_byte_boundary(orc):
    """Hidden widths 33, 65, 17 and 3 samples per worker: a group's window of an activation starts 6 x 33 x 4 bytes into
    the tensor, which is no multiple of 16, so the 128-bit elementwise kernels must take their element-wise path."""
    net = sy.Net("mlp-ragged", sy.mlp_layers([70, 33, 65, 17, 5]), [4], 1, 1, 70, 5, 4, 3, 0.05, "fp32")
    run_parity(orc, net, 3 * net.K, param_tol=1e-5, loss_tol=1e-5, worker_groups=2)


def test_fp32_vgg_with_biases_grouped_matches_oracle(orc):
    layers, starts = sy.vgg_layers(widths=(6, 10, 12, 20), in_c=3, classes=10)
    net = sy.Net("vgg-small", layers, starts[1:], 16, 16, 3, 10, 4, 3, 0.05, "fp32")
    run_parity(orc, net, 3 * net.K, param_tol=1e-5, loss_tol=1e-5, grad_tol=0.2, grad_best_tol=1e-5, worker_groups=4)


def test_bf16_tensor_core_resnet_grouped_matches_oracle(orc):
    net = _tensor_core_net()
    run_parity(orc, net, 3 * net.K, grad_tol=2e-2, noise_factor=3.0, loss_tol=1e-2, worker_groups=2)


@pytest.mark.parametrize("groups", [2, 4])
def test_bf16_grouped_run_equals_ungrouped_run_up_to_summation_order(groups):
    import torch
    from paper_2509_05679_b200 import binding
    net = _tensor_core_net()
    p0 = sy.perturb_params(sy.init_params(net.layers, 0, bf16=True), net.layers, 7, 0.1)
    runs = []
    for g in (1, groups):
        ctx = make_ctx(net, p0, worker_groups=g)
        launches0 = ctx.stats()[1]
        grads = None
        for t in range(2 * net.K):
            x, y = binding.to_device("bf16", sy.batch_inputs(net, t)), torch.from_numpy(sy.batch_labels(net, t)).cuda()
            ctx.step(x, y)
            ctx.wait_ingest()
            if t == 2 * net.K - 2:
                grads = ctx.grads()          # first step in which every module has a gradient
        runs.append((ctx.params(), grads, ctx.stats()[1] - launches0))
        ctx.close()
    (p1, g1, n1), (pg, gg, ng) = runs
    assert ng > n1, "the grouped context launched no more kernels than the ungrouped one: grouping did not happen"
    scale = np.sqrt(np.mean(g1.astype(np.float64) ** 2))
    assert np.max(np.abs(gg - g1)) <= 1e-3 * scale, "first full gradient differs by more than fp32 summation order"
    assert np.max(np.abs(pg - p1)) <= 1e-3 * np.max(np.abs(p1))
