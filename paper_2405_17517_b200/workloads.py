"""Seeded synthetic populations shaped like the WASH paper's workloads.

Holds only shapes and random inputs -- none of the method's arithmetic -- so that the
GPU library's tests, the CPU oracle's tests and the benchmark can all draw the same
inputs from one place.  The paper trains ResNet-18 / ResNet-50 / VGG-16 populations of
N in {3, 5, 10} with SGD momentum ("Experimental setup"); no dataset or trained weight
is needed here, only the learnable-tensor tables of those networks.  BatchNorm running
statistics are not part of a stack ("Training methods": they are neither permuted nor
recomputed), so the tables list learnable tensors only.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import numpy as np

Table = List[Tuple[str, Tuple[int, ...]]]

ALIGN_ELEMS = 8  # tensors start on a multiple of 8 elements in a stack row


def _conv_bn(table: Table, name: str, cout: int, cin: int, k: int) -> None:
    table.append((name + ".conv.weight", (cout, cin, k, k)))
    table.append((name + ".bn.weight", (cout,)))
    table.append((name + ".bn.bias", (cout,)))


def resnet18_table(num_classes: int = 100) -> Table:
    """ResNet-18 for small images: 3x3 stem, four stages of two basic blocks."""
    t: Table = []
    _conv_bn(t, "stem", 64, 3, 3)
    cin = 64
    for stage, cout in enumerate((64, 128, 256, 512)):
        for block in range(2):
            name = "layer%d.%d" % (stage + 1, block)
            _conv_bn(t, name + ".a", cout, cin, 3)
            _conv_bn(t, name + ".b", cout, cout, 3)
            if block == 0 and cin != cout:
                _conv_bn(t, name + ".shortcut", cout, cin, 1)
            cin = cout
    t.append(("fc.weight", (num_classes, 512)))
    t.append(("fc.bias", (num_classes,)))
    return t


def resnet50_table(num_classes: int = 1000) -> Table:
    """ResNet-50: 7x7 stem, bottleneck stages [3, 4, 6, 3], expansion 4."""
    t: Table = []
    _conv_bn(t, "stem", 64, 3, 7)
    cin = 64
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for block in range(blocks):
            name = "layer%d.%d" % (stage + 1, block)
            _conv_bn(t, name + ".a", width, cin, 1)
            _conv_bn(t, name + ".b", width, width, 3)
            _conv_bn(t, name + ".c", width * 4, width, 1)
            if block == 0:
                _conv_bn(t, name + ".downsample", width * 4, cin, 1)
            cin = width * 4
    t.append(("fc.weight", (num_classes, 2048)))
    t.append(("fc.bias", (num_classes,)))
    return t


def flat_table(P: int) -> Table:
    return [("flat", (int(P),))]


def numels(table: Table) -> np.ndarray:
    return np.array([int(np.prod(shape)) for _, shape in table], dtype=np.int64)


def padded_offsets(numel: Sequence[int], align: int = ALIGN_ELEMS):
    """Element offset of every tensor in a stack row and the row length."""
    offs, cur = [], 0
    for d in numel:
        offs.append(cur)
        cur += (int(d) + align - 1) // align * align
    return np.array(offs, dtype=np.int64), int(cur)


def _tensor_std(name: str, shape: Tuple[int, ...]) -> float:
    if len(shape) >= 2:  # conv / linear weight: Kaiming normal, fan_out mode
        fan_out = shape[0] * int(np.prod(shape[2:])) if len(shape) > 2 else shape[0]
        return math.sqrt(2.0 / fan_out)
    return 0.02  # scale used only for the per-model perturbation of 1-D tensors


def init_population(table: Table, N: int, seed: int, drift: float = 0.1) -> np.ndarray:
    """Dense [N, P] float32 population: a shared Kaiming-style initialisation theta_0
    (the paper starts every model from the same point, Algorithm 1) plus a per-model
    perturbation of `drift` x the tensor's scale, standing in for a few steps of
    training, so that every exchange is visible in the output."""
    rng = np.random.default_rng(seed)
    sizes = numels(table)
    P = int(sizes.sum())
    out = np.empty((N, P), dtype=np.float32)
    pos = 0
    for (name, shape), d in zip(table, sizes):
        d = int(d)
        std = _tensor_std(name, shape)
        if len(shape) >= 2:
            base = rng.standard_normal(d, dtype=np.float32) * np.float32(std)
        elif name.endswith("bn.weight"):
            base = np.ones(d, dtype=np.float32)
        else:
            base = np.zeros(d, dtype=np.float32)
        noise = rng.standard_normal((N, d), dtype=np.float32) * np.float32(drift * std)
        out[:, pos:pos + d] = base[None, :] + noise
        pos += d
    return out


def init_momentum(table: Table, N: int, seed: int, scale: float = 1e-3) -> np.ndarray:
    rng = np.random.default_rng(seed)
    P = int(numels(table).sum())
    return rng.standard_normal((N, P), dtype=np.float32) * np.float32(scale)


def flat_population(N: int, P: int, seed: int = 0, std: float = 0.05) -> np.ndarray:
    """N x P values drawn N(0, std^2), every model distinct."""
    rng = np.random.default_rng(seed)
    return rng.standard_normal((N, P), dtype=np.float32) * np.float32(std)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), by torch's own conversion."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def to_stack(dense: np.ndarray, numel: Sequence[int], offset: Sequence[int], padded_P: int,
             layout: int = 0, pad_value=None) -> np.ndarray:
    """Place a dense [N, P] array into a padded stack: [N][padded_P] (layout 0) or
    [padded_P][N] (layout 1).  Padding elements get `pad_value` (default: a NaN /
    0xFFFF pattern that any accidental use would expose)."""
    N = dense.shape[0]
    if pad_value is None:
        pad_value = np.float32(np.nan) if dense.dtype == np.float32 else dense.dtype.type(0xFFFF)
    row = np.full((N, int(padded_P)), pad_value, dtype=dense.dtype)
    pos = 0
    for d, off in zip(numel, offset):
        d, off = int(d), int(off)
        row[:, off:off + d] = dense[:, pos:pos + d]
        pos += d
    return np.ascontiguousarray(row if layout == 0 else row.T)


def from_stack(stack: np.ndarray, N: int, numel: Sequence[int], offset: Sequence[int], padded_P: int,
               layout: int = 0) -> np.ndarray:
    """Inverse of to_stack: the dense [N, P] logical view (a copy)."""
    row = stack.reshape(N, padded_P) if layout == 0 else stack.reshape(padded_P, N).T
    return np.concatenate([row[:, int(o):int(o) + int(d)] for d, o in zip(numel, offset)], axis=1) \
        if len(numel) else np.zeros((N, 0), dtype=stack.dtype)


# The five benchmark configurations (shapes only).
CONFIGS = {
    "cfg1_flat_n3": dict(N=3, table="flat:1048576", p=0.01, schedule=None, dtype="f32", opt=False),
    "cfg2_resnet18_n5": dict(N=5, table="resnet18:100", p=0.001, schedule=None, dtype="f32", opt=True),
    "cfg3_resnet50_n10": dict(N=10, table="resnet50:1000", p=0.01, schedule="decreasing", dtype="f32", opt=True),
    "cfg4_resnet50_bf16_n8": dict(N=8, table="resnet50:1000", p=0.005, schedule=None, dtype="bf16", opt=True),
}


def table_from_spec(spec: str) -> Table:
    kind, arg = spec.split(":")
    if kind == "flat":
        return flat_table(int(arg))
    if kind == "resnet18":
        return resnet18_table(int(arg))
    if kind == "resnet50":
        return resnet50_table(int(arg))
    raise ValueError(spec)
