"""fdg_bias_grad_static -- the bias-gradient reduction for callers that may not allocate device memory
(plug-ins inside another framework's memory pool, loops that cannot afford the device-wide
synchronisation of cudaMalloc/cudaFree, processes with a fixed memory budget).

The check: the training step computes bias gradients with the same reduction, using scratch from the
context's allocator; its result comes back through fdg_step + fdg_grads.  For a one-layer network with
zero weights the error gradient that reduction sees is known in closed form,
dY = (1/classes - onehot(labels)) / M, so the test rebuilds dY, hands it to the static entry point and
compares the two bias gradients -- on two calls in a row with different labels, so that a value left
in the shared scratch array by the first call would show up in the second.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.  It needs nothing from them and also passes alone in a fresh process."""
import numpy as np
import pytest

from paper_2509_05679_b200 import synth as sy

pytestmark = pytest.mark.gpu

CLASSES, FEATURES, WORKERS, BATCH = 10, 24, 2, 48
M = WORKERS * BATCH


def rel_err(a, b):
    b = np.asarray(b, np.float64)
    floor = 0.1 * np.sqrt(np.mean(b * b)) + 1e-30
    return float(np.max(np.abs(np.asarray(a, np.float64) - b) / np.maximum(np.abs(b), floor)))


def closed_form_dy(labels):
    """What the step's softmax cross-entropy produces for all-zero logits, in fp32."""
    p = np.exp(-np.log(np.float32(CLASSES), dtype=np.float32), dtype=np.float32)
    dy = np.full((M, CLASSES), p, dtype=np.float32)
    dy[np.arange(M), labels] -= np.float32(1.0)
    return dy * np.float32(1.0 / M)


def test_static_bias_gradient_matches_the_training_step_twice_in_a_row():
    import torch
    from paper_2509_05679_b200 import binding

    layers = [(sy.LINEAR, FEATURES, CLASSES, 1, sy.FLAG_BIAS)]
    ctx = binding.Context(layers, [], WORKERS, BATCH, 0.0, dtype="fp32", in_shape=(1, 1, FEATURES), num_classes=CLASSES)
    ctx.set_params(np.zeros(ctx.n_params, np.float32))          # zero weights, lr 0: logits stay zero
    out = torch.empty(CLASSES, dtype=torch.float32, device="cuda")
    rng = np.random.default_rng(7)
    for call in range(2):
        x = rng.standard_normal((M, FEATURES)).astype(np.float32)
        labels = rng.integers(0, CLASSES, M).astype(np.int32)
        ctx.step(binding.to_device("fp32", x), torch.from_numpy(labels).cuda(), want_loss=True)
        db_step = ctx.grads()[-CLASSES:]                         # existing entry points: fdg_step + fdg_grads
        dy = torch.from_numpy(closed_form_dy(labels)).cuda()
        out.fill_(float("nan"))
        torch.cuda.synchronize()
        binding.bias_grad_static(dy, "fp32", M, CLASSES, out)    # default stream; no allocation inside
        torch.cuda.synchronize()
        db_static = out.cpu().numpy()
        assert np.isfinite(db_static).all()
        assert rel_err(db_static, db_step) <= 1e-5, (call, db_static, db_step)
        counts = np.bincount(labels, minlength=CLASSES)
        assert rel_err(db_static, 0.1 - counts / M) <= 1e-5      # and both equal the closed form
    ctx.close()


def test_static_entry_point_bf16_ragged_rows_and_rejected_sizes():
    import torch
    from paper_2509_05679_b200 import binding

    rng = np.random.default_rng(3)
    rows, ch = 1000 + 37, 200                                     # spans several chunks, ragged tail, > 128 channels
    a = sy.round_to_bf16(rng.standard_normal((rows, ch)).astype(np.float32))
    out = torch.empty(ch, dtype=torch.float32, device="cuda")
    for _ in range(2):
        binding.bias_grad_static(torch.from_numpy(a).cuda().to(torch.bfloat16), "bf16", rows, ch, out)
        torch.cuda.synchronize()
        assert rel_err(out.cpu().numpy(), a.astype(np.float64).sum(0)) <= 1e-5
    with pytest.raises(binding.FdgError) as e:                    # beyond the fixed scratch: refused, nothing launched
        binding.bias_grad_static(out, "fp32", 4, 4097, out)
    assert e.value.status == 1 and "4096" in str(e.value)
    with pytest.raises(binding.FdgError):
        binding.bias_grad_static(out, "fp32", 0, 8, out)
