"""GPU parity: the CUDA library against the oracle, through the C ABI, on seeded workloads."""
import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu

ALL_FLAGS = [0, B.TEAM_F_DCD, B.TEAM_F_LAC, B.TEAM_F_DCD | B.TEAM_F_LAC]


@pytest.fixture(scope="module")
def weights_cache():
    cache = {}

    def get(shape):
        key = (shape.hidden, shape.n_experts, shape.inter, shape.n_shared, shape.dtype, shape.seed)
        if key not in cache:
            cache[key] = W.make_weights(shape)
        return cache[key]
    return get


@pytest.mark.parametrize("flags", ALL_FLAGS)
def test_c1_tiny_fp32_all_steps(flags, weights_cache):
    stats = P.run_schedule(W.C1, weights_cache(W.C1), W.make_schedule(W.C1), flags)
    assert len(stats) == 8 and all(s["exact"] for s in stats)
    assert max(s["rel_err"] for s in stats) <= P.TOL_F32


@pytest.mark.parametrize("flags", ALL_FLAGS)
@pytest.mark.parametrize("shape", [W.MINI_BF16, W.MINI_SHARED, W.MINI_WRAP], ids=lambda s: s.name)
def test_mini_bf16_tensor_path(shape, flags, weights_cache):
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags)
    assert all(s["launches"] == 3 for s in stats)


@pytest.mark.parametrize("shape", [W.MINI_BF16, W.MINI_SHARED], ids=lambda s: s.name)
def test_mini_bf16_fma_diagnostic_path(shape, weights_cache):
    P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), 3, force_simt=True)


@pytest.mark.parametrize("flags", [0, 1, 3])
def test_c2_sdar_shape(flags, weights_cache):
    stats = P.run_schedule(W.C2, weights_cache(W.C2), W.make_schedule(W.C2), flags)
    assert len(stats) == 4
    if flags == 3:
        assert [s["rows"] for s in stats] == [4, 4, 3, 2]


@pytest.mark.parametrize("flags", [0, 3])
def test_c3_llada_shape_with_shared_expert(flags, weights_cache):
    stats = P.run_schedule(W.C3, weights_cache(W.C3), W.make_schedule(W.C3), flags)
    assert len(stats) == 8


@pytest.mark.parametrize("seqs", [1, 4, 16, 64])
def test_c4_batch_sweep(seqs, weights_cache):
    shape = W.c4(seqs)
    steps = W.make_schedule(shape)
    # all four steps for the small batches, two for the large ones (the oracle takes seconds per step there)
    steps = steps if seqs <= 4 else steps[1:3]
    P.run_schedule(shape, weights_cache(shape), steps, 3)
    if seqs <= 4:
        P.run_schedule(shape, weights_cache(shape), steps, 0)
