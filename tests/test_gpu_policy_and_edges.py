"""GPU parity for the policy knobs and the degenerate steps the C ABI exposes, and for the two named
calls team_route and team_select_experts on their own.

Every case goes through the C ABI and is compared with the oracle row by row (tests/_parity.py).  The
readings exercised here are the ones the paper leaves open: Eq. 4 as printed ("<") against the wording of
Sec. 5.1 ("no more than L_h positions away"), whether the previous block's last token counts as decoded
at a block's first step, routing weights with and without renormalisation over the k chosen, and the
steps Sec. 4.1 produces at the end of a block (every row cached).
"""
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

# resident streaming kernel / gather streaming kernel / tensor-memory kernel with a shared expert / fp32 kernels
KNOB_SHAPES = [W.C2, W.STREAM_GATHER, W.MINI_SHARED, W.C1]


def _weights(shape, cache={}):
    key = (shape.hidden, shape.n_experts, shape.inter, shape.n_shared, shape.dtype, shape.seed)
    if key not in cache:
        cache[key] = W.make_weights(shape)
    return cache[key]


def _classes(stats):
    return np.concatenate([s["classes"] for s in stats])


@pytest.mark.parametrize("knob", [dict(hot_dist_inclusive=0), dict(prefix_decoded=0), dict(norm_topk=0),
                                  dict(hot_dist_inclusive=0, prefix_decoded=0, norm_topk=0)],
                         ids=["eq4_strict_less", "no_prefix", "unnormalised", "all_three"])
@pytest.mark.parametrize("shape", KNOB_SHAPES, ids=lambda s: s.name)
def test_policy_knobs(shape, knob):
    steps = W.make_schedule(shape)
    stats = P.run_schedule(shape, _weights(shape), steps, TEAM, **knob)
    assert len(stats) == len(steps)
    if "hot_dist_inclusive" in knob or "prefix_decoded" in knob:
        # the knob must move at least one row between hot and cold somewhere in the schedule, or the case tests nothing
        dcfg = P.oracle_config(shape, TEAM)
        default = np.concatenate([O.classify(dcfg, s["tok_state"], s["conf"], s["pos"], s["group"], s["branch"])
                                  for s in steps])
        assert (_classes(stats) != default).any(), "this schedule does not exercise the knob"


@pytest.mark.parametrize("shape", [W.C2, W.MINI_SHARED, W.C1], ids=lambda s: s.name)
def test_empty_first_round_falls_back_to_free_routing(shape):
    """First step of a block with no decoded prefix and no confident token: Eq. 4 makes every row cold, Algorithm 1's
    first round is empty, and all masked rows of such a group are routed freely.  With two groups, the second one
    keeps a newly accepted token, so fallback and regular groups sit in one call."""
    step = {k: np.array(v, copy=True) for k, v in W.make_schedule(shape)[0].items()}
    step["tok_state"][:] = W.TOK_MASKED                    # (speculative branches accept a token of their own at step 0)
    step["conf"][:] = 0.1
    if shape.seqs > 1:
        first_of_g1 = int(np.flatnonzero(step["group"] == 1)[0])
        step["tok_state"][first_of_g1] = W.TOK_NEW
        step["conf"][first_of_g1] = 1.0
    stats = P.run_schedule(shape, _weights(shape), [step], TEAM, prefix_decoded=0)
    cls = stats[0]["classes"]
    g0 = step["group"] == 0
    assert (cls[g0] == O.CLS_FIRST).all()                  # the fallback
    if shape.seqs > 1:
        assert (cls[~g0] == O.CLS_COLD).any()              # the regular group still has cold rows


@pytest.mark.parametrize("shape", [W.C2, W.STREAM_GATHER, W.C1], ids=lambda s: s.name)
def test_step_with_every_row_cached(shape):
    """The last steps of a block under delayed caching (Sec. 4.1): nothing is computed, y keeps the previous step's
    values, no expert is activated, and the status word stays clean.  A regular step follows on the same context."""
    steps = W.make_schedule(shape)
    cached = {k: np.array(v, copy=True) for k, v in steps[-1].items()}
    cached["tok_state"][:] = W.TOK_CACHED
    cached["conf"][:] = 1.0
    stats = P.run_schedule(shape, _weights(shape), [steps[1], cached, cached, steps[2]], TEAM)
    for s in stats[1:3]:
        assert s["rows"] == 0 and s["n_active"] == 0
    assert stats[3]["rows"] > 0 and stats[3]["n_active"] >= shape.top_k
    # with delayed caching off the same rows are all computed (a decoded row is a first-round row)
    stats = P.run_schedule(shape, _weights(shape), [cached], B.TEAM_F_LAC)
    assert stats[0]["rows"] == shape.rows


@pytest.mark.parametrize("shape", [W.C2, W.MINI_BF16, W.C1], ids=lambda s: s.name)
def test_single_row_call(shape):
    one = dataclasses.replace(shape, name=shape.name + "_t1", block=1, n_steps=3, unmask_per_step=1, unmask_every=1)
    steps = W.make_schedule(one)
    assert steps[0]["x"].shape[0] == 1
    for flags in (0, TEAM):
        stats = P.run_schedule(one, _weights(shape), steps, flags)
        assert [s["rows"] for s in stats] == ([1, 1, 1] if flags == 0 else [1, 1, 0])
        assert all(s["n_active"] == (shape.top_k + shape.n_shared if s["rows"] else 0) for s in stats)


@pytest.mark.parametrize("switch", [dict(flags=0), dict(flags=B.TEAM_F_DCD), dict(L_hot=0, tau_hot=0.99),
                                    dict(hot_dist_inclusive=0, norm_topk=0)],
                         ids=["to_vanilla", "lac_off", "nothing_hot", "strict_unnormalised"])
def test_policy_switch_between_steps_of_one_context(switch):
    """team_set_policy between two steps: the following steps run under the new policy, on the same context."""
    for shape in (W.C2, W.MINI_SHARED):
        steps = W.make_schedule(shape)
        stats = P.run_schedule(shape, _weights(shape), steps, TEAM, policy_switch=(2, switch))
        assert len(stats) == len(steps)
        if switch.get("flags", TEAM) & B.TEAM_F_DCD == 0:
            assert all(s["rows"] == shape.rows for s in stats[2:])


@pytest.mark.parametrize("tables", [True, False], ids=["with_tables", "choices_only"])
@pytest.mark.parametrize("shape", [W.C2, W.MINI_SHARED, W.C1], ids=lambda s: s.name)
def test_periodic_refresh(shape, tables):
    """Refresh-N (Sec. 4.1, second paragraph; Table 3): every N-th step recomputes all tokens, the others run with
    delayed caching.  With N = 2 the steps 0, 2, 4 compute every row."""
    steps = W.make_schedule(shape)
    stats = P.run_schedule(shape, _weights(shape), steps, TEAM, tables=tables, refresh_every=2)
    plain = P.run_schedule(shape, _weights(shape), steps, TEAM, tables=tables)
    for s, q in zip(stats, plain):
        assert s["rows"] == (shape.rows if s["step"] % 2 == 0 else q["rows"])
    assert any(s["rows"] > q["rows"] for s, q in zip(stats, plain))       # the schedule does have cached rows to refresh


def _plain_topk_reference(ocfg, logits32, probs, cls_computed):
    """Plain (unrestricted) top-k, weights and margin of every computed row, from the oracle's pieces."""
    T = logits32.shape[0]
    idx = np.full((T, ocfg.top_k), -1, dtype=np.int32)
    w = np.zeros((T, ocfg.top_k))
    margin = np.full(T, np.inf)
    for t in np.flatnonzero(cls_computed):
        take, margin[t] = O.topk_row(logits32[t], ocfg.top_k)
        idx[t] = take
        w[t] = O.routing_weights(probs[t], take, ocfg.norm_topk)
    return idx, w, margin


@pytest.mark.parametrize("flags", [0, TEAM])
@pytest.mark.parametrize("shape", [W.C2, W.MINI_SHARED, W.C1, W.c4(4), W.C3], ids=lambda s: s.name)
def test_route_then_select_against_the_oracle(shape, flags):
    """The two named calls on their own: team_route's softmax table, plain top-k, weights and margin against the
    oracle's router and top-k; then team_select_experts on the same context against the oracle's selection, all
    twelve tables."""
    weights = _weights(shape)
    ocfg = P.oracle_config(shape, flags)
    layer = P.Layer(shape, weights, flags)
    try:
        for si, step in enumerate(W.make_schedule(shape)[:4]):
            T = step["x"].shape[0]
            what = f"{shape.name} flags={flags} step={si}"
            x_dev = B.to_device(step["x"], P.dtype_code(shape))
            st = B.state_to_device(step)
            out = B.alloc_routing(layer.cfg, T)
            for name in ("probs", "topk_w", "margin"):
                out[name].fill_(-7.0)
            out["topk_idx"].fill_(-7)
            B.team_route(layer.ctx, x_dev, st, out)
            assert B.team_last_launch_count(layer.ctx) == 2
            torch.cuda.synchronize()
            got = {n: out[n].cpu().numpy() for n in ("probs", "topk_idx", "topk_w", "margin")}
            logits32, probs = O.router(step["x"], weights["w_router"])
            computed = np.zeros(T, dtype=bool)
            computed[O.active_rows(step["tok_state"], flags)] = True
            idx, w, margin = _plain_topk_reference(ocfg, logits32, probs, computed)
            np.testing.assert_allclose(got["probs"][computed], probs[computed], rtol=0, atol=P.PROBS_ATOL, err_msg=what)
            assert not got["probs"][~computed].any() and (got["topk_idx"][~computed] == -1).all()
            assert not got["topk_w"][~computed].any() and np.isinf(got["margin"][~computed]).all()
            n_pinned = 0
            for t in np.flatnonzero(computed):
                if P.ordering_margin(logits32[t], idx[t], range(shape.n_experts)) <= P.MARGIN:
                    assert set(got["topk_idx"][t].tolist()) <= set(range(shape.n_experts))
                    continue
                n_pinned += 1
                np.testing.assert_array_equal(got["topk_idx"][t], idx[t], err_msg=f"{what} row {t}")
                np.testing.assert_allclose(got["topk_w"][t], w[t], atol=2e-6, rtol=1e-5, err_msg=what)
                if np.isinf(margin[t]):
                    assert np.isinf(got["margin"][t])
                else:
                    assert abs(got["margin"][t] - margin[t]) < 1e-5
            assert n_pinned >= int(P.MIN_PINNED_FRACTION * computed.sum())

            out2 = B.alloc_routing(layer.cfg, T)
            B.team_select_experts(layer.ctx, st, out2)
            code, detail = B.team_read_status(layer.ctx)
            assert code == B.TEAM_OK, (code, detail)
            got2 = B.routing_to_host(out2)
            ref = O.select_experts(ocfg, logits32, probs, step["tok_state"], step["conf"], step["pos"], step["group"],
                                   step["branch"])
            ref["logits"], ref["probs"] = logits32, probs
            exact, pin = P.compare_routing(ocfg, ref, got2, step["group"], what, return_pin=True)
            assert pin.sum() >= int(P.MIN_PINNED_FRACTION * T)
    finally:
        layer.close()
