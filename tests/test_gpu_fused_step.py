"""GPU parity of the one-kernel step: with at most 8 rows per call and no dispatch table asked for,
team_moe_forward runs router, selection (Eq. 4, Algorithm 1's two rounds) and the experts as a single
cooperative kernel whose CTAs meet at a grid barrier between the router and the selection.  The cases ask
for the rows' choices only, so that this is the path that runs, and compare everything it exports and every
computed output row with the oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu

TEAM = B.TEAM_F_DCD | B.TEAM_F_LAC
# SDAR shape; several passes per CTA and a shared expert; 128 slots over 258 experts (two router rows per CTA)
SHAPES = [W.C2, W.STREAM_MULTI, W.STREAM_WIDE]


def _weights(shape, cache={}):
    key = (shape.hidden, shape.n_experts, shape.inter, shape.n_shared, shape.dtype, shape.seed)
    if key not in cache:
        cache[key] = W.make_weights(shape)
    return cache[key]


@pytest.mark.parametrize("flags", [0, B.TEAM_F_DCD, B.TEAM_F_LAC, TEAM])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: s.name)
def test_one_kernel_step_against_the_oracle(shape, flags):
    stats = P.run_schedule(shape, _weights(shape), W.make_schedule(shape), flags, tables=False)
    assert all(s["launches"] == 1 for s in stats)
    if shape is W.C2 and flags == TEAM:
        assert [s["rows"] for s in stats] == [4, 4, 3, 2]


@pytest.mark.parametrize("knob", [dict(hot_dist_inclusive=0), dict(prefix_decoded=0), dict(norm_topk=0)],
                         ids=["eq4_strict_less", "no_prefix", "unnormalised"])
def test_one_kernel_step_policy_knobs(knob):
    for shape in (W.C2, W.STREAM_MULTI):
        stats = P.run_schedule(shape, _weights(shape), W.make_schedule(shape), TEAM, tables=False, **knob)
        assert all(s["launches"] == 1 for s in stats)


def test_one_kernel_step_degenerate_steps():
    """Empty first round (fallback to free routing), a step with every row cached, a single row."""
    shape = W.C2
    steps = W.make_schedule(shape)
    cold = {k: np.array(v, copy=True) for k, v in steps[0].items()}
    cold["tok_state"][:] = W.TOK_MASKED
    cold["conf"][:] = 0.1
    stats = P.run_schedule(shape, _weights(shape), [cold], TEAM, tables=False, prefix_decoded=0)
    assert (stats[0]["classes"] == O.CLS_FIRST).all()
    cached = {k: np.array(v, copy=True) for k, v in steps[-1].items()}
    cached["tok_state"][:] = W.TOK_CACHED
    stats = P.run_schedule(shape, _weights(shape), [steps[1], cached, cached, steps[2]], TEAM, tables=False)
    assert [s["rows"] for s in stats][1:3] == [0, 0] and all(s["launches"] == 1 for s in stats)
    one = dataclasses.replace(shape, name="c2_t1", block=1, n_steps=3, unmask_per_step=1, unmask_every=1)
    stats = P.run_schedule(one, _weights(shape), W.make_schedule(one), TEAM, tables=False)
    assert [s["rows"] for s in stats] == [1, 1, 0]


def test_three_kernel_sequence_is_still_there_and_agrees():
    """The diagnostic knob keeps router, selection and experts as separate launches; same exports, same y."""
    shape = W.C2
    stats = P.run_schedule(shape, _weights(shape), W.make_schedule(shape), TEAM, tables=False,
                           knobs=[(B.TEAM_KNOB_NO_FUSE, 1)])
    assert all(s["launches"] == 3 for s in stats)


def test_policy_switch_and_weight_switch_on_one_context():
    shape = W.C2
    P.run_schedule(shape, _weights(shape), W.make_schedule(shape), TEAM, tables=False, policy_switch=(2, dict(flags=0)))


def test_barrier_wait_runs_out_and_reports_a_timeout_without_hanging():
    """The grid barrier's wait is bounded.  With the diagnostic knob that makes it wait for an arrival that never
    comes and a limit of 200 microseconds, every CTA gives up, the kernel returns, the status word reads
    TEAM_ERR_TIMEOUT, and the context works normally afterwards."""
    shape = W.C2
    weights = _weights(shape)
    layer = P.Layer(shape, weights, TEAM)
    try:
        step = W.make_schedule(shape)[1]
        T = step["x"].shape[0]
        x_dev, st = B.to_device(step["x"], B.TEAM_DTYPE_BF16), B.state_to_device(step)
        y = torch.zeros((T, shape.hidden), dtype=torch.float32, device="cuda")
        B.team_debug_knob(layer.ctx, B.TEAM_KNOB_WAIT_LIMIT_US, 200)
        B.team_debug_knob(layer.ctx, B.TEAM_KNOB_EXTRA_ARRIVALS, 1)
        B.team_moe_forward(layer.ctx, x_dev, st, None, y)
        code, detail = B.team_read_status(layer.ctx)
        assert code == B.TEAM_ERR_TIMEOUT and detail == 20
        assert B.team_read_status(layer.ctx)[0] == B.TEAM_OK          # reading cleared it
        B.team_debug_knob(layer.ctx, B.TEAM_KNOB_EXTRA_ARRIVALS, 0)
        B.team_debug_knob(layer.ctx, B.TEAM_KNOB_WAIT_LIMIT_US, 1000000)
        out = {n: v for n, v in B.alloc_routing(layer.cfg, T).items() if n in P.CHOICE_TABLES}
        B.team_moe_forward(layer.ctx, x_dev, st, out, y)
        assert B.team_read_status(layer.ctx)[0] == B.TEAM_OK
        ocfg = P.oracle_config(shape, TEAM)
        y_ref, ref = O.moe_forward(ocfg, weights, step["x"], step["tok_state"], step["conf"], step["pos"],
                                   step["group"], step["branch"])
        comp = ref["tok_class"] != O.CLS_SKIP
        err = np.abs(y.cpu().numpy()[comp] - y_ref[comp]).max()
        assert err <= P.TOL_BF16 * np.abs(y_ref[comp]).max()
    finally:
        layer.close()
