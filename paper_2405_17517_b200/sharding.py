"""Host-side planning of coordinate shards for several GPUs.

The shuffle's random draws are keyed by the global (tensor, coordinate), so a population
can be cut anywhere along its coordinates: every rank holds all N models' values of its
own coordinates, runs the same kernels through wash_create_segments, and the union of the
ranks' results equals the single-GPU result bit for bit -- no communication in the data
path.  This module only decides who owns which coordinates.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

Segment = Tuple[int, int, int]   # (tensor index, first coordinate within the tensor, coordinates)


def plan_shards(numel: Sequence[int], world_size: int) -> List[List[Segment]]:
    """Cut the concatenated coordinates of the tensors into world_size contiguous shares
    of (almost) equal size.  A cut inside a tensor is moved down to a multiple of 4
    coordinates, because four neighbouring coordinates share one Philox block and one
    16-byte load.  Returns, per rank, its segments in order; a rank may get none when there
    are fewer groups of coordinates than ranks."""
    if world_size < 1:
        raise ValueError("world_size must be at least 1")
    sizes = [int(d) for d in numel]
    if any(d <= 0 for d in sizes):
        raise ValueError("tensor sizes must be positive")
    total = sum(sizes)
    starts = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    cuts = []
    for r in range(world_size + 1):
        pos = total * r // world_size
        t = int(np.searchsorted(starts, pos, side="right") - 1)
        t = min(t, len(sizes) - 1)
        local = pos - int(starts[t])
        if r == world_size:
            cuts.append(total)
        else:
            cuts.append(int(starts[t]) + (local // 4) * 4)
    plans: List[List[Segment]] = []
    for r in range(world_size):
        lo, hi = cuts[r], cuts[r + 1]
        segs: List[Segment] = []
        for t, d in enumerate(sizes):
            a, b = max(lo, int(starts[t])), min(hi, int(starts[t]) + d)
            if a < b:
                segs.append((t, a - int(starts[t]), b - a))
        plans.append(segs)
    return plans


def segment_arrays(segments: Sequence[Segment]):
    """(numel, tensor_id, coord_begin) arrays as wash_create_segments takes them."""
    numel = np.array([s[2] for s in segments], dtype=np.int64)
    tensor_id = np.array([s[0] for s in segments], dtype=np.uint32)
    coord_begin = np.array([s[1] for s in segments], dtype=np.int64)
    return numel, tensor_id, coord_begin


def segment_probs(p_layer: Sequence[float], segments: Sequence[Segment]) -> np.ndarray:
    """Per-segment probabilities from per-tensor (per-layer) ones."""
    return np.array([float(p_layer[s[0]]) for s in segments], dtype=np.float64)


def dense_slices(numel: Sequence[int], segments: Sequence[Segment]) -> List[slice]:
    """Column ranges of a dense [N, P] array (tensors concatenated) that a shard owns."""
    starts = np.concatenate([[0], np.cumsum([int(d) for d in numel])]).astype(np.int64)
    return [slice(int(starts[t]) + c0, int(starts[t]) + c0 + cnt) for t, c0, cnt in segments]
