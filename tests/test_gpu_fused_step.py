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


def _ys_of_a_schedule(shape, steps, knobs, host_entry=False):
    """y after every step of a schedule on a fresh context (no exports: the one-kernel step)."""
    layer = P.Layer(shape, _weights(shape), TEAM)
    for knob, value in knobs:
        B.team_debug_knob(layer.ctx, knob, value)
    T, H = shape.rows, shape.hidden
    y = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    y_host = torch.zeros((T, H), dtype=torch.float32)
    out = []
    try:
        for step in steps:
            if host_entry:
                st_host = {"tok_state": torch.as_tensor(step["tok_state"].astype(np.uint8)),
                           "conf": torch.as_tensor(step["conf"].astype(np.float32)),
                           "pos": torch.as_tensor(step["pos"].astype(np.int32)),
                           "group": torch.as_tensor(step["group"].astype(np.int32)),
                           "branch": torch.as_tensor(step["branch"].astype(np.int32))}
                B.team_moe_forward_host(layer.ctx, torch.as_tensor(step["x"]).to(torch.bfloat16), st_host, None, y_host)
                out.append(y_host.clone())
            else:
                B.team_moe_forward(layer.ctx, B.to_device(step["x"], B.TEAM_DTYPE_BF16), B.state_to_device(step), None, y)
                assert B.team_last_launch_count(layer.ctx) == 1
                out.append(y.cpu())
        assert B.team_read_status(layer.ctx)[0] == B.TEAM_OK
    finally:
        layer.close()
    return out


@pytest.mark.parametrize("shape", [W.C2, W.STREAM_MULTI], ids=lambda s: s.name)
def test_ordered_combine_is_reproducible_bit_for_bit(shape):
    """With the ordered combine the contributions to y are summed in a fixed order: two runs, and the host-buffer
    entry point against the device one, give identical bits; the default mode (fp32 reductions in arrival order)
    agrees with it to rounding of the sums; and the ordered result matches the oracle like any other."""
    steps = W.make_schedule(shape) * 2
    ordered = [(B.TEAM_KNOB_ORDERED_COMBINE, 1)]
    a = _ys_of_a_schedule(shape, steps, ordered)
    b = _ys_of_a_schedule(shape, steps, ordered)
    c = _ys_of_a_schedule(shape, steps, ordered, host_entry=True)
    d = _ys_of_a_schedule(shape, steps, [])
    for ya, yb, yc, yd in zip(a, b, c, d):
        assert torch.equal(ya, yb) and torch.equal(ya, yc)
        assert torch.allclose(ya, yd, rtol=0, atol=1e-5 * float(ya.abs().max()))
    stats = P.run_schedule(shape, _weights(shape), W.make_schedule(shape), TEAM, tables=False, knobs=ordered)
    assert all(s["launches"] == 1 for s in stats)
