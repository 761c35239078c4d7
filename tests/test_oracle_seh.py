"""Pins for the decode-loop oracle (threshold acceptance, speculative branches, chained verification)."""
import json
import os

import numpy as np
import pytest

from oracle import seh_oracle as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = json.load(open(os.path.join(ROOT, "tests", "golden", "seh_decode_cases.json")))


@pytest.mark.parametrize("case", GOLD["cases"], ids=lambda c: c["name"])
def test_hand_derived_cases(case):
    tau = GOLD["tau"]
    pred, conf = np.array(case["pred"], dtype=np.int32), np.array(case["conf"], dtype=np.float32)
    assert S.verify_chain(pred, conf, case["spec_pos"], case["spec_tok"], tau) == case["chain"]
    token, state, sp, stok, adopted, newly = S.seh_step(case["token"], case["state"], case["spec_pos"], case["spec_tok"],
                                                        pred, conf, tau)
    assert adopted == case["adopted"] and newly == case["newly"]
    assert token.tolist() == case["token_after"] and state.tolist() == case["state_after"]
    assert sp.tolist() == case["spec_pos_after"] and stok.tolist() == case["spec_tok_after"]


def _random_step(rng, L=8, vocab=5):
    state = rng.integers(0, 3, L).astype(np.uint8)
    token = np.where(state == S.TOK_MASKED, -1, rng.integers(0, vocab, L)).astype(np.int32)
    masked = np.flatnonzero(state == S.TOK_MASKED)
    spec_pos = np.full(2, -1, np.int32)
    spec_tok = np.full(2, -1, np.int32)
    picks = rng.permutation(masked)[:rng.integers(0, 3)]
    for i, p in enumerate(picks):
        spec_pos[i], spec_tok[i] = p, rng.integers(0, vocab)
    pred = rng.integers(0, vocab, (4, L)).astype(np.int32)
    conf = np.where(rng.random((4, L)) < 0.5, rng.uniform(0.951, 1.0, (4, L)), rng.uniform(0, 0.95, (4, L))).astype(np.float32)
    return token, state, spec_pos, spec_tok, pred, conf


def test_invariants_over_random_steps():
    """Whatever the inputs: the base branch's acceptance (Eq. 3) is always part of the result; with nothing confirmed
    it is the whole result; accepted tokens turn NEW and earlier NEW tokens cached; decoded positions never change;
    candidates are masked positions ordered by the adopted branch's confidence."""
    rng = np.random.default_rng(3)
    seen_chains = set()
    for _ in range(3000):
        token, state, spec_pos, spec_tok, pred, conf = _random_step(rng)
        tau = 0.95
        t2, s2, sp2, st2, adopted, newly = S.seh_step(token, state, spec_pos, spec_tok, pred, conf, tau)
        chain = S.verify_chain(pred, conf, spec_pos, spec_tok, tau)
        seen_chains.add(tuple(chain))
        base = [p for p in range(len(state)) if state[p] == S.TOK_MASKED and conf[0][p] > np.float32(tau)]
        assert set(base) <= set(newly)
        for p in base:
            assert t2[p] == pred[0][p]
        if chain == [0]:
            assert newly == base and adopted == 0
        for p in range(len(state)):
            if state[p] != S.TOK_MASKED:
                assert t2[p] == token[p] and s2[p] == S.TOK_CACHED
            elif p in newly:
                assert s2[p] == S.TOK_NEW and t2[p] >= 0
            else:
                assert s2[p] == S.TOK_MASKED and t2[p] == -1
        left = [p for p in range(len(state)) if s2[p] == S.TOK_MASKED]
        want = sorted(left, key=lambda p: (-float(conf[adopted][p]), p))[:2] + [-1, -1]
        assert sp2.tolist() == want[:2]
        for i in range(2):
            assert st2[i] == (pred[adopted][sp2[i]] if sp2[i] >= 0 else -1)
    assert {(0,), (0, 1), (0, 2), (0, 1, 3), (0, 2, 3)} <= seen_chains


def test_rows_of_the_next_forward_pass():
    """Branch 0 carries the base states, branch 1 marks the 1st candidate as accepted, branch 2 the 2nd, branch 3
    both (Sec. 5.4); the confidence handed to Eq. 4 is 1 for decoded positions."""
    state = np.array([2, 1, 0, 0, 0], np.uint8)
    rows = S.next_rows(state, [3, 2], np.array([1, 1, 0.8, 0.9, 0.1], np.float32), seq=7)
    ts = np.array(rows["tok_state"]).reshape(4, 5)
    assert ts[0].tolist() == [2, 1, 0, 0, 0] and ts[1].tolist() == [2, 1, 0, 1, 0]
    assert ts[2].tolist() == [2, 1, 1, 0, 0] and ts[3].tolist() == [2, 1, 1, 1, 0]
    cf = np.array(rows["conf"]).reshape(4, 5)
    assert cf[0].tolist() == pytest.approx([1, 1, 0.8, 0.9, 0.1]) and cf[3].tolist() == pytest.approx([1, 1, 1, 1, 0.1])
    assert rows["branch"] == [b for b in range(4) for _ in range(5)] and set(rows["group"]) == {7}
    assert rows["pos"] == list(range(5)) * 4


def test_a_scripted_block_by_hand():
    """Four positions; the script confirms the 1st candidate at the second forward pass.  Speculation finishes the
    block in 3 forward passes (TPF 4/3); threshold decoding alone (Eq. 3) needs 4 (TPF 1)."""
    L, tau = 4, 0.95
    truth = [5, 6, 7, 8]
    pred = np.tile(np.array(truth, np.int32), (4, 4, 1))                    # [steps][branch][pos]: always the right token
    conf = np.zeros((4, 4, L), np.float32)
    conf[0, :, :] = [0.99, 0.80, 0.30, 0.10]        # pass 1: position 0 accepted; candidates 1 (0.80), 2 (0.30)
    conf[1, 0, :] = [1.00, 0.97, 0.50, 0.20]        # pass 2, base: candidate 1 confirmed
    conf[1, 1, :] = [1.00, 1.00, 0.96, 0.30]        #         branch 1 (1 decoded): position 2 now confident
    conf[1, 2, :] = [1.00, 0.90, 1.00, 0.30]
    conf[1, 3, :] = [1.00, 1.00, 1.00, 0.40]        #         branch 3 is trusted too (2 confirmed in branch 1): nothing more
    conf[2, :, :] = [1.00, 1.00, 1.00, 0.99]        # pass 3: the last position
    conf[3, :, :] = 1.0
    rec, fwd, acc = S.decode_block(pred, conf, L, tau)
    assert [r["newly"] for r in rec] == [[0], [1, 2], [3]] and [r["adopted"] for r in rec] == [0, 3, 1]      # (pass 3: the one candidate left is confirmed by the base branch)
    assert (fwd, acc) == (3, 4)
    conf_v = conf.copy()
    conf_v[2, :, :] = [1.0, 1.0, 0.97, 0.30]        # without the branches position 2 is only reached at pass 3
    conf_v[3, :, :] = [1.0, 1.0, 1.0, 0.99]
    rec, fwd, acc = S.decode_block(pred, conf_v, L, tau, speculate=False)
    assert [r["newly"] for r in rec] == [[0], [1], [2], [3]] and (fwd, acc) == (4, 4)
