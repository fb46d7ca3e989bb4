"""The shared library loads without a GPU and exports what include/wash.h declares;
host-only entry points behave; argument errors are caught before any device work."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import build as wash_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    wash_build.build()
    return B.load()


def _declared_functions():
    with open(os.path.join(ROOT, "include", "wash.h")) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\(", " ".join(
        ln for ln in text.splitlines() if not ln.lstrip().startswith("#")))) - {"defined"})


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"wash_create", "wash_shuffle", "wash_shuffle_opt_state", "wash_shuffle_both", "papa_ema",
            "population_average", "wash_step_host"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_has_the_same_names(lib):
    for name in _declared_functions():
        assert hasattr(B, name), name


def test_layer_probs_match_the_oracle_and_reject_bad_input(lib):
    for L in (1, 2, 5, 62, 161):
        for sched in (0, 1, 2):
            assert np.array_equal(B.wash_layer_probs(L, 0.01, sched), oracle.layer_probs(L, 0.01, sched))
    for args in ((0, 0.1, 0), (3, 1.5, 0), (3, float("nan"), 0), (3, 0.1, 7)):
        with pytest.raises(B.WashError) as e:
            B.wash_layer_probs(*args)
        assert e.value.code == B.WASH_ERR_ARG


def test_create_rejects_bad_arguments_before_touching_a_device(lib):
    for N, numel, kw in ((1, [8], {}), (65, [8], {}), (3, [], {}), (3, [0], {}), (3, [1 << 32], {}),
                         (3, [8], dict(layout=2)), (3, [8], dict(coord_begin=[2])),
                         (3, [8], dict(coord_begin=[(1 << 32) - 4]))):
        with pytest.raises(B.WashError) as e:
            B.wash_create_segments(N, numel, kw.get("tensor_id"), kw.get("coord_begin"), kw.get("layout", 0), 0)
        assert e.value.code == B.WASH_ERR_ARG, (N, numel, kw)
    assert "must be" in B.wash_last_error() or "coord_begin" in B.wash_last_error()


def test_null_context_is_an_argument_error(lib):
    assert lib.wash_destroy(None) == B.WASH_ERR_ARG
    assert lib.wash_shuffle(None, 0, 0.5, None, 0, None, None) == B.WASH_ERR_ARG
    assert lib.papa_ema(None, 0, ctypes.c_float(0.5), None) == B.WASH_ERR_ARG
    assert lib.wash_launch_count() == 0 or lib.wash_launch_count() > 0
