"""Seeded synthetic workloads: layer lists, parameter layout, inputs, labels, initial weights.

This module is the only code shared by the CUDA path's callers and the CPU oracle's callers.
It holds no arithmetic of the training method itself: it describes networks (as plain layer
lists), enumerates the canonical parameter order, and draws random numbers from numpy's
counter-based Philox generator.

Layer records are 5 integers ``(kind, c_in, c_out, stride, flags)``.

Canonical parameter order (both the library and the oracle use it): layers in list order; for
each layer ``W`` then ``b`` (linear ``W[out][in]``; conv ``W[c_out][kh][kw][c_in]``), batch-norm
``gamma`` then ``beta``; a residual add with projection carries ``Wp[c_out][c_in]`` (1x1 conv,
no bias) followed by the projection batch-norm's ``gamma`` and ``beta``.

Activations are NHWC, worker-major: rows ``s*B .. (s+1)*B-1`` of a batch belong to worker ``s``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np

# layer kinds (values are part of the C interface)
LINEAR, CONV3X3, CONV1X1, RELU, MAXPOOL2, GLOBAL_AVGPOOL, BATCHNORM, RES_BEGIN, RES_ADD = range(9)
FLAG_BIAS = 1        # LINEAR / CONV*: layer has a bias vector
FLAG_PROJ = 1        # RES_ADD: shortcut is conv1x1(stride) + batch-norm instead of identity

Layer = Tuple[int, int, int, int, int]


@dataclass
class Net:
    """A network plus the way it is split and fed (one benchmark configuration)."""
    name: str
    layers: List[Layer]
    splits: List[int]            # first layer index of modules 2..K (K-1 entries)
    in_h: int
    in_w: int
    in_c: int
    classes: int
    n_workers: int
    batch: int                   # per-worker batch B
    lr: float
    dtype: str                   # "fp32" or "bf16"
    steps: int = 20
    extra: dict = field(default_factory=dict)

    @property
    def K(self) -> int:
        return len(self.splits) + 1

    @property
    def M(self) -> int:
        return self.n_workers * self.batch

    @property
    def in_elems(self) -> int:
        return self.in_h * self.in_w * self.in_c


def param_shapes(layers: Sequence[Layer]) -> List[Tuple[int, str, Tuple[int, ...], int]]:
    """[(layer index, tensor name, shape, fan_in)] in canonical order."""
    out = []
    for i, (kind, cin, cout, stride, flags) in enumerate(layers):
        if kind == LINEAR:
            out.append((i, "W", (cout, cin), cin))
            if flags & FLAG_BIAS:
                out.append((i, "b", (cout,), 0))
        elif kind in (CONV3X3, CONV1X1):
            r = 3 if kind == CONV3X3 else 1
            out.append((i, "W", (cout, r, r, cin), r * r * cin))
            if flags & FLAG_BIAS:
                out.append((i, "b", (cout,), 0))
        elif kind == BATCHNORM:
            out.append((i, "gamma", (cin,), -1))
            out.append((i, "beta", (cin,), 0))
        elif kind == RES_ADD and (flags & FLAG_PROJ):
            out.append((i, "Wp", (cout, 1, 1, cin), cin))
            out.append((i, "gamma_p", (cout,), -1))
            out.append((i, "beta_p", (cout,), 0))
    return out


def param_count(layers: Sequence[Layer]) -> int:
    return int(sum(int(np.prod(s)) for _, _, s, _ in param_shapes(layers)))


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even); returns fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def init_params(layers: Sequence[Layer], seed: int = 0, bf16: bool = False) -> np.ndarray:
    """He-normal weights (std = sqrt(2 / fan_in)), zero biases, gamma = 1, beta = 0; fp32."""
    g = _rng(seed)
    parts = []
    for _, _, shape, fan_in in param_shapes(layers):
        n = int(np.prod(shape))
        if fan_in > 0:
            parts.append((g.standard_normal(n) * np.sqrt(2.0 / fan_in)).astype(np.float32))
        elif fan_in == -1:
            parts.append(np.ones(n, dtype=np.float32))
        else:
            parts.append(np.zeros(n, dtype=np.float32))
    p = np.concatenate(parts) if parts else np.zeros(0, np.float32)
    return round_to_bf16(p) if bf16 else p


def perturb_params(params: np.ndarray, layers: Sequence[Layer], seed: int, scale: float = 0.1) -> np.ndarray:
    """Make biases / gamma / beta non-trivial so that tests exercise them (fp32)."""
    g = _rng(seed)
    p = params.copy()
    off = 0
    for _, _, shape, fan_in in param_shapes(layers):
        n = int(np.prod(shape))
        if fan_in <= 0:
            p[off:off + n] += (g.standard_normal(n) * scale).astype(np.float32)
        off += n
    return p


def batch_inputs(net: Net, t: int, stream: int = 0) -> np.ndarray:
    """Inputs of iteration t: [M, in_h, in_w, in_c] i.i.d. N(0,1), fp32 (bf16-representable
    when the configuration computes in bf16).  `stream` selects an independent data stream."""
    x = _rng(1000 + t + 1000003 * stream).standard_normal((net.M, net.in_h, net.in_w, net.in_c)).astype(np.float32)
    return round_to_bf16(x) if net.dtype == "bf16" else x


def batch_labels(net: Net, t: int, stream: int = 0) -> np.ndarray:
    """Labels of iteration t: int32[M], uniform in 0..classes-1."""
    return _rng(2000 + t + 1000003 * stream).integers(0, net.classes, size=net.M, dtype=np.int32)


# ----------------------------------------------------------------------------- networks

def mlp_layers(sizes: Sequence[int]) -> List[Layer]:
    layers: List[Layer] = []
    for i in range(len(sizes) - 1):
        layers.append((LINEAR, sizes[i], sizes[i + 1], 1, FLAG_BIAS))
        if i < len(sizes) - 2:
            layers.append((RELU, sizes[i + 1], sizes[i + 1], 1, 0))
    return layers


def vgg_layers(widths=(64, 128, 256, 512), in_c=3, classes=10) -> Tuple[List[Layer], List[int]]:
    """conv,conv,pool per width (no pool after the last pair), global avgpool, FC.
    Returns (layers, first-layer index of every conv pair) so callers can derive splits."""
    layers: List[Layer] = []
    starts = []
    c = in_c
    for i, w in enumerate(widths):
        starts.append(len(layers))
        for _ in range(2):
            layers.append((CONV3X3, c, w, 1, FLAG_BIAS))
            layers.append((RELU, w, w, 1, 0))
            c = w
        if i < len(widths) - 1:
            layers.append((MAXPOOL2, c, c, 2, 0))
    layers.append((GLOBAL_AVGPOOL, c, c, 1, 0))
    layers.append((LINEAR, c, classes, 1, FLAG_BIAS))
    return layers, starts


def resnet_layers(widths=(64, 128, 256, 512), blocks=2, in_c=3, classes=10):
    """3x3 stem + basic-block stages (stride 1,2,2,2) + global avgpool + FC, batch-norm after
    every conv, 1x1-conv + batch-norm projection where the shape changes.
    Returns (layers, first-layer index of every basic block)."""
    layers: List[Layer] = []
    block_starts = []
    layers += [(CONV3X3, in_c, widths[0], 1, 0), (BATCHNORM, widths[0], widths[0], 1, 0),
               (RELU, widths[0], widths[0], 1, 0)]
    c = widths[0]
    for si, w in enumerate(widths):
        for bi in range(blocks):
            stride = 2 if (si > 0 and bi == 0) else 1
            block_starts.append(len(layers))
            proj = FLAG_PROJ if (stride != 1 or c != w) else 0
            layers += [(RES_BEGIN, c, c, 1, 0),
                       (CONV3X3, c, w, stride, 0), (BATCHNORM, w, w, 1, 0), (RELU, w, w, 1, 0),
                       (CONV3X3, w, w, 1, 0), (BATCHNORM, w, w, 1, 0),
                       (RES_ADD, c, w, stride, proj), (RELU, w, w, 1, 0)]
            c = w
    layers += [(GLOBAL_AVGPOOL, c, c, 1, 0), (LINEAR, c, classes, 1, FLAG_BIAS)]
    return layers, block_starts


def config(idx: int, *, n_workers: int | None = None, batch: int | None = None,
           width_div: int = 1, K: int | None = None) -> Net:
    """The five benchmark configurations (idx 0..4). ``n_workers`` / ``batch`` / ``width_div``
    shrink a configuration for parity tests without changing its structure."""
    if idx == 0:
        layers = mlp_layers([3072, 512, 256, 10])
        net = Net("C1-mlp-fp32", layers, [2], 1, 1, 3072, 10, 2, 32, 0.01, "fp32", steps=20)
    elif idx == 1:
        h = 1024 // width_div
        layers = mlp_layers([3072] + [h] * 8 + [10])
        # linear layer j (0-based) sits at list index 2j; modules hold layers (1,2)(3,4)(5,6)(7,8,9)
        net = Net("C2-mlp-bf16", layers, [4, 8, 12], 1, 1, 3072, 10, 4, 128, 0.05, "bf16", steps=200)
    elif idx == 2:
        widths = tuple(w // width_div for w in (64, 128, 256, 512))
        layers, starts = vgg_layers(widths)
        # step size 0.005: the configuration names none, and at 0.05 this network (eight convolutions, no normalisation)
        # diverges under the stale gradients within ten iterations in any arithmetic
        net = Net("C3-vgg-bf16", layers, starts[1:], 32, 32, 3, 10, 4, 128, 0.005, "bf16", steps=50)
    elif idx in (3, 4):
        widths = tuple(w // width_div for w in (64, 128, 256, 512))
        layers, bs = resnet_layers(widths)
        if idx == 3:
            splits = [bs[2], bs[4], bs[6]]           # stage boundaries; stem with stage 1
            net = Net("C4-resnet18-K4-bf16", layers, splits, 32, 32, 3, 10, 8, 128, 0.05, "bf16", steps=50)
        else:
            splits = bs[1:]                          # one basic block per module
            net = Net("C5-resnet18-K8-bf16", layers, splits, 32, 32, 3, 10, 16, 256, 0.05, "bf16", steps=50)
    elif idx in (5, 6):
        # the paper's experiment shape (Sec. 5) on synthetic data: ResNet-20 (3 stages of 16/32/64 channels, 3 blocks
        # each), 4 data-groups, mini-batch 194 read as the total (48 samples per worker), step size 0.1;
        # 5: traditional backpropagation (K = 1), 6: decoupled into K = 2 modules (cut between blocks 4 and 5)
        layers, bs = resnet_layers(widths=(16, 32, 64), blocks=3)
        net = Net("resnet20-S4-K1-fp32" if idx == 5 else "resnet20-S4-K2-fp32", layers, [] if idx == 5 else [bs[4]],
                  32, 32, 3, 10, 4, 48, 0.1, "fp32", steps=50)
    else:
        raise ValueError("config index 0..6")
    if K is not None and K == 1:
        net.splits = []
    if n_workers is not None:
        net.n_workers = n_workers
    if batch is not None:
        net.batch = batch
    return net


def without_relu(net: Net) -> Net:
    """The same network with every ReLU layer taken out (split points re-indexed).  Its gradients have no
    kinks, which makes it the deep network on which two bf16 evaluations can be compared tensor by tensor."""
    keep = [i for i, l in enumerate(net.layers) if l[0] != RELU]
    new_index = {old: new for new, old in enumerate(keep)}
    return Net(net.name + "-relu-free", [net.layers[i] for i in keep], [new_index[s] for s in net.splits], net.in_h, net.in_w,
               net.in_c, net.classes, net.n_workers, net.batch, net.lr, net.dtype, net.steps, dict(net.extra))


def flops_per_sample(net: Net) -> float:
    """Algorithmic FLOPs per sample per step: forward 2*MACs, backward dgrad + wgrad, minus the
    first weighted layer's dgrad (nothing consumes it)."""
    h, w = net.in_h, net.in_w
    fwd = []
    for kind, cin, cout, stride, flags in net.layers:
        if kind == LINEAR:
            fwd.append(2.0 * cin * cout)
            h = w = 1
        elif kind in (CONV3X3, CONV1X1):
            r = 9 if kind == CONV3X3 else 1
            h, w = h // stride, w // stride
            fwd.append(2.0 * r * cin * cout * h * w)
        elif kind == MAXPOOL2:
            h, w = h // 2, w // 2
        elif kind == GLOBAL_AVGPOOL:
            h = w = 1
        elif kind == RES_ADD and (flags & FLAG_PROJ):
            fwd.append(2.0 * cin * cout * h * w)
    return 3.0 * sum(fwd) - fwd[0]
