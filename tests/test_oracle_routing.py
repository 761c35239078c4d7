"""Pins for the oracle's router, top-k, classification, selection and dispatch.

Each test checks the oracle against something other than itself: brute-force
enumeration, closed forms, library routines, hand-derived truth tables, or the
structural properties the paper states.
"""
import itertools
import json
import os

import numpy as np
import pytest
import scipy.special

from oracle import team_oracle as O
from paper_2602_08404_b200 import workloads as W


def _rand_logits(rng, T, E):
    return rng.standard_normal((T, E)).astype(np.float32)


# --- router ---------------------------------------------------------------
def test_router_matches_library_softmax_and_plain_dot():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 24)).astype(np.float32)
    wr = (0.3 * rng.standard_normal((7, 24))).astype(np.float32)
    logits32, probs = O.router(x, wr)
    # plain triple loop in Python floats (fp64), independent of numpy matmul
    for t in range(5):
        for e in range(7):
            acc = 0.0
            for h in range(24):
                acc += float(x[t, h]) * float(wr[e, h])
            assert logits32[t, e] == np.float32(acc)
    ref = scipy.special.softmax(logits32.astype(np.float64), axis=1)
    np.testing.assert_allclose(probs, ref, rtol=1e-13, atol=0)
    np.testing.assert_allclose(probs.sum(axis=1), 1.0, rtol=1e-13)


def test_router_closed_forms():
    # equal scores -> uniform; a transposed operand or a wrong axis breaks this
    x = np.ones((3, 8), dtype=np.float32)
    wr = np.ones((5, 8), dtype=np.float32)
    logits32, probs = O.router(x, wr)
    assert np.all(logits32 == 8.0)
    np.testing.assert_allclose(probs, 0.2, rtol=1e-15)
    # one-hot rows pick out a column of the router matrix
    x = np.eye(4, dtype=np.float32)
    wr = np.arange(12, dtype=np.float32).reshape(3, 4)
    logits32, _ = O.router(x, wr)
    np.testing.assert_array_equal(logits32, wr.T)
    # two experts: softmax is the logistic function of the score difference
    x = np.array([[1.0, 2.0]], dtype=np.float32)
    wr = np.array([[0.5, 0.25], [-1.0, 0.5]], dtype=np.float32)
    l, p = O.router(x, wr)
    d = float(l[0, 0]) - float(l[0, 1])
    assert abs(p[0, 0] - 1.0 / (1.0 + np.exp(-d))) < 1e-15


# --- top-k ----------------------------------------------------------------
@pytest.mark.parametrize("E,k", [(16, 2), (8, 3), (10, 1), (6, 6)])
def test_topk_is_the_argmax_subset_by_enumeration(E, k):
    rng = np.random.default_rng(E * 10 + k)
    for _ in range(20):
        l = _rand_logits(rng, 1, E)[0]
        p = scipy.special.softmax(l.astype(np.float64))
        take, margin = O.topk_row(l, k)
        best = max(itertools.combinations(range(E), k), key=lambda s: sum(p[list(s)]))
        assert set(take) == set(best)
        assert list(take) == sorted(take, key=lambda e: -l[e])       # descending order
        rest = [l[e] for e in range(E) if e not in take]
        if rest:
            assert margin == pytest.approx(float(min(l[take])) - float(max(rest)))
            assert margin >= 0
        else:
            assert margin == float("inf")


def test_topk_restricted_by_enumeration_and_ties():
    rng = np.random.default_rng(5)
    E, k = 12, 3
    for _ in range(20):
        l = _rand_logits(rng, 1, E)[0]
        allowed = set(rng.choice(E, size=5, replace=False).tolist())
        take, _ = O.topk_row(l, k, allowed=allowed)
        best = max(itertools.combinations(sorted(allowed), k), key=lambda s: sum(l[list(s)]))
        assert set(take) == set(best) and set(take) <= allowed
    # ties go to the lower expert id
    l = np.array([1.0, 3.0, 3.0, 3.0, 0.0], dtype=np.float32)
    assert O.topk_row(l, 2)[0] == [1, 2]
    assert O.topk_row(l, 2)[1] == 0.0
    assert O.topk_row(l, 2, allowed={0, 2, 3, 4})[0] == [2, 3]


def test_routing_weights_sum_to_one_and_full_k_is_softmax():
    rng = np.random.default_rng(7)
    l = _rand_logits(rng, 1, 9)[0]
    p = scipy.special.softmax(l.astype(np.float64))
    take, _ = O.topk_row(l, 4)
    w = O.routing_weights(p, take, 1)
    assert abs(w.sum() - 1.0) < 1e-15
    assert np.all(np.diff(w) <= 0)
    np.testing.assert_allclose(w, p[take] / p[take].sum(), rtol=1e-15)
    take, _ = O.topk_row(l, 9)
    np.testing.assert_allclose(O.routing_weights(p, take, 1), p[take], rtol=1e-14)
    np.testing.assert_allclose(O.routing_weights(p, take[:3], 0), p[take[:3]], rtol=0)


# --- classification (Eq. 4) -------------------------------------------------
def _golden_cases(golden_dir):
    with open(os.path.join(golden_dir, "eq4_classification.json")) as f:
        return json.load(f)["cases"]


def test_classification_truth_tables(golden_dir):
    code = {"M": O.TOK_MASKED, "N": O.TOK_NEW, "C": O.TOK_CACHED}
    out = {O.CLS_SKIP: "S", O.CLS_FIRST: "F", O.CLS_COLD: "C"}
    cases = _golden_cases(golden_dir)
    assert len(cases) >= 10
    for c in cases:
        T = len(c["states"])
        cfg = O.Config(hidden=1, n_experts=4, top_k=1, inter=1, flags=c["flags"],
                       tau_hot=c["tau_hot"], L_hot=c["L_hot"],
                       hot_dist_inclusive=c["hot_dist_inclusive"],
                       prefix_decoded=c["prefix_decoded"])
        st = [code[ch] for ch in c["states"]]
        cls = O.classify(cfg, st, c["conf"], c.get("pos", list(range(T))),
                         c.get("group", [0] * T), c.get("branch", [0] * T))
        assert "".join(out[v] for v in cls) == c["expect"], c["name"]


def test_classification_limits():
    rng = np.random.default_rng(3)
    T = 12
    st = rng.integers(0, 3, size=T)
    conf = rng.uniform(0, 1, size=T).astype(np.float32)
    pos, grp, br = np.arange(T), np.zeros(T, int), np.zeros(T, int)
    base = dict(hidden=1, n_experts=4, top_k=1, inter=1, flags=O.F_DCD | O.F_LAC, prefix_decoded=1)
    # L_h >= block length, or tau_h below every confidence: nothing is cold
    for cfg in (O.Config(L_hot=T, tau_hot=0.7, **base), O.Config(L_hot=0, tau_hot=-1.0, **base)):
        cls = O.classify(cfg, st, conf, pos, grp, br)
        assert not np.any(cls == O.CLS_COLD)
        np.testing.assert_array_equal(cls == O.CLS_SKIP, st == O.TOK_CACHED)


# --- selection (Algorithm 1) and dispatch -----------------------------------
def _random_case(seed, T=12, E=16, k=2, flags=3, ns=0, groups=1, L_hot=1):
    rng = np.random.default_rng(seed)
    cfg = O.Config(hidden=8, n_experts=E, top_k=k, inter=4, n_shared=ns, flags=flags,
                   tau_hot=0.7, L_hot=L_hot, max_groups=groups)
    logits = _rand_logits(rng, T, E)
    probs = scipy.special.softmax(logits.astype(np.float64), axis=1)
    per = T // groups
    st = np.zeros(T, dtype=np.uint8)
    for g in range(groups):
        n_dec = rng.integers(0, per)
        st[g * per:g * per + n_dec] = O.TOK_CACHED
        if n_dec:
            st[g * per + n_dec - 1] = O.TOK_NEW
    conf = rng.uniform(0, 0.95, size=T).astype(np.float32)
    pos = np.tile(np.arange(per), groups)
    grp = np.repeat(np.arange(groups), per)
    br = np.zeros(T, dtype=int)
    return cfg, logits, probs, st, conf, pos, grp, br


@pytest.mark.parametrize("seed", range(12))
def test_selection_by_brute_force_on_tiny_inputs(seed):
    cfg, logits, probs, st, conf, pos, grp, br = _random_case(seed, groups=1 + seed % 2)
    r = O.select_experts(cfg, logits, probs, st, conf, pos, grp, br)
    E, k = cfg.n_experts, cfg.top_k
    cls = r["tok_class"]
    for g in range(cfg.max_groups):
        first = [t for t in range(len(st)) if grp[t] == g and cls[t] == O.CLS_FIRST]
        # E_A(g): union over first-round rows of the best-k subset found by enumeration
        ea = set()
        for t in first:
            ea |= set(max(itertools.combinations(range(E), k), key=lambda s: sum(probs[t, list(s)])))
        bits = {e for e in range(E) if (int(r["group_mask"][g, e // 64]) >> (e % 64)) & 1}
        assert bits == ea and len(ea) >= k
        for t in range(len(st)):
            if grp[t] != g:
                continue
            if cls[t] == O.CLS_COLD:
                best = max(itertools.combinations(sorted(ea), k), key=lambda s: sum(probs[t, list(s)]))
                assert set(r["topk_idx"][t]) == set(best)
            if cls[t] != O.CLS_SKIP:
                assert abs(r["topk_w"][t].sum() - 1.0) < 1e-12
                np.testing.assert_allclose(
                    r["topk_w"][t], probs[t, r["topk_idx"][t]] / probs[t, r["topk_idx"][t]].sum(), rtol=1e-13)
            else:
                assert np.all(r["topk_idx"][t] == -1) and np.all(r["topk_w"][t] == 0)


@pytest.mark.parametrize("seed", range(8))
def test_structural_properties_of_the_activated_set(seed):
    cfg, logits, probs, st, conf, pos, grp, br = _random_case(seed + 100, T=16, E=32, k=4, groups=2)
    team = O.select_experts(cfg, logits, probs, st, conf, pos, grp, br)
    van_cfg = O.Config(**{**cfg.__dict__, "flags": 0})
    van = O.select_experts(van_cfg, logits, probs, st, conf, pos, grp, br)
    # TEAM disabled: activated set is the union of every row's plain top-k
    union = set()
    for t in range(16):
        union |= set(np.argsort(-probs[t], kind="stable")[:4].tolist())
    assert set(van["active"].tolist()) == union
    assert van["n_rows_active"] == 16 and not np.any(van["tok_class"] == O.CLS_COLD)
    # TEAM's set is contained in the vanilla set; cold rows add no expert
    assert set(team["active"].tolist()) <= union
    first_union = set()
    for t in range(16):
        if team["tok_class"][t] == O.CLS_FIRST:
            first_union |= set(team["topk_idx"][t].tolist())
    assert set(team["active"].tolist()) == first_union
    # rows computed = masked + newly accepted (delayed caching)
    assert team["n_rows_active"] == int(np.sum(st != O.TOK_CACHED))
    # if the necessary set is everything, the second round equals the first
    full = O.Config(**{**cfg.__dict__, "top_k": 32})
    # (k = E makes every first-round row contribute all experts)
    r_full = O.select_experts(full, logits, probs, st, conf, pos, grp, br)
    for t in range(16):
        if r_full["tok_class"][t] != O.CLS_SKIP:
            assert sorted(r_full["topk_idx"][t].tolist()) == list(range(32))


def test_cold_rows_equal_free_routing_when_their_choice_is_already_necessary():
    # A cold row whose own top-k lies inside E_A must keep exactly its own top-k.
    cfg, logits, probs, st, conf, pos, grp, br = _random_case(4, T=10, E=8, k=2)
    st[:] = O.TOK_MASKED
    st[0] = O.TOK_NEW
    conf[:] = 0.1
    logits[:] = logits[0]                      # every row routes like row 0
    probs = scipy.special.softmax(logits.astype(np.float64), axis=1)
    r = O.select_experts(cfg, logits, probs, st, conf, pos, grp, br)
    assert np.sum(r["tok_class"] == O.CLS_COLD) > 0
    for t in range(10):
        np.testing.assert_array_equal(r["topk_idx"][t], r["topk_idx"][0])
    assert r["n_active"] == 2


@pytest.mark.parametrize("ns", [0, 1, 2])
def test_dispatch_tables(ns):
    cfg, logits, probs, st, conf, pos, grp, br = _random_case(9 + ns, T=12, E=16, k=3, ns=ns)
    r = O.select_experts(cfg, logits, probs, st, conf, pos, grp, br)
    T, E, k = 12, 16, 3
    rows = [t for t in range(T) if r["tok_class"][t] != O.CLS_SKIP]
    S = len(rows) * (k + ns)
    assert r["expert_count"].sum() == S
    assert r["expert_offset"][0] == 0 and r["expert_offset"][-1] == S
    np.testing.assert_array_equal(np.diff(r["expert_offset"]), r["expert_count"])
    perm = r["perm"][:S]
    assert np.all(r["perm"][S:] == -1)
    # expected slot ids and the expert of each slot, then a library stable sort
    slot_ids, slot_exp = [], []
    for t in rows:
        for j in range(k):
            slot_ids.append(t * k + j)
            slot_exp.append(int(r["topk_idx"][t, j]))
    for s in range(ns):
        for t in rows:
            slot_ids.append(T * k + s * T + t)
            slot_exp.append(E + s)
    slot_ids, slot_exp = np.array(slot_ids), np.array(slot_exp)
    order = np.lexsort((slot_ids, slot_exp))
    np.testing.assert_array_equal(perm, slot_ids[order])
    assert sorted(perm.tolist()) == sorted(slot_ids.tolist())
    np.testing.assert_array_equal(r["active"], np.flatnonzero(r["expert_count"] > 0))
    for sid in perm:
        t, w = O.slot_row_weight(cfg, T, int(sid), r["topk_w"])
        assert t in rows
        if sid >= T * k:
            assert w == 1.0


def test_schedule_rows_follow_delayed_caching():
    # scripted schedule of the SDAR-shaped block: one token accepted per step
    steps = W.make_schedule(W.C2)
    expect_active = [4, 4, 3, 2]     # masked + newly accepted at steps 0..3
    for s, step in enumerate(steps):
        assert len(O.active_rows(step["tok_state"], O.F_DCD)) == expect_active[s]
        assert len(O.active_rows(step["tok_state"], 0)) == 4
