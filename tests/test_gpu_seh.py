"""GPU parity of the decode-loop glue (team_seh_step) against the oracle: whole blocks decoded step by step from a
scripted language-model head, every state array and every row of the next forward pass compared bit for bit; and
the rows fed into team_moe_forward."""
import numpy as np
import pytest
import torch

from oracle import seh_oracle as S
from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu
TAU = 0.95


def _decode_blocks_both(n_seqs, L, n_branches, seed, max_steps=80):
    pred, conf = W.make_decode_script(n_seqs, L, max_steps, seed, n_branches=n_branches)
    state, rows = B.seh_alloc(n_seqs, L, n_branches)
    adopted = torch.zeros(n_seqs, dtype=torch.int32, device="cuda")
    B.team_seh_step(n_seqs, L, n_branches, TAU, state, None, None, rows, adopted)         # begin the block
    o_tok = [np.full(L, -1, np.int32) for _ in range(n_seqs)]
    o_st = [np.zeros(L, np.uint8) for _ in range(n_seqs)]
    o_sp = [np.array([-1, -1], np.int32) for _ in range(n_seqs)]
    o_stk = [np.array([-1, -1], np.int32) for _ in range(n_seqs)]
    o_fwd, o_acc = np.zeros(n_seqs, int), np.zeros(n_seqs, int)

    def check_rows(conf_adopted):
        got = {n: v.cpu().numpy().reshape(n_seqs, -1) for n, v in rows.items()}
        for s in range(n_seqs):
            want = S.next_rows(o_st[s], o_sp[s] if n_branches == 4 else [-1, -1], conf_adopted[s], s)
            for n in got:
                w = np.array(want[n]).reshape(4, L)[:n_branches].reshape(-1)
                np.testing.assert_array_equal(got[n][s], w.astype(got[n].dtype), err_msg=f"rows {n} seq {s}")

    check_rows([np.zeros(L, np.float32)] * n_seqs)
    chains = set()
    for step in range(max_steps):
        if all((st != S.TOK_MASKED).all() for st in o_st):
            break
        p4 = np.zeros((n_seqs, 4, L), np.int32)
        c4 = np.zeros((n_seqs, 4, L), np.float32)
        p4[:, :n_branches], c4[:, :n_branches] = pred[step], conf[step]
        B.team_seh_step(n_seqs, L, n_branches, TAU, state, torch.as_tensor(pred[step]).cuda().contiguous(),
                        torch.as_tensor(conf[step]).cuda().contiguous(), rows, adopted)
        conf_adopted = []
        for s in range(n_seqs):
            done = (o_st[s] != S.TOK_MASKED).all()
            o_tok[s], o_st[s], o_sp[s], o_stk[s], ad, newly = S.seh_step(o_tok[s], o_st[s], o_sp[s], o_stk[s], p4[s], c4[s], TAU)
            if n_branches == 1:
                o_sp[s][:], o_stk[s][:] = -1, -1
            chains.add(ad)
            o_fwd[s] += 1
            o_acc[s] += len(newly)
            conf_adopted.append(c4[s][ad])
            assert int(adopted[s]) == ad, (step, s)
            assert not (done and newly)
        np.testing.assert_array_equal(state["token"].cpu().numpy(), np.stack(o_tok))
        np.testing.assert_array_equal(state["state"].cpu().numpy(), np.stack(o_st))
        np.testing.assert_array_equal(state["spec_pos"].cpu().numpy(), np.stack(o_sp))
        np.testing.assert_array_equal(state["spec_tok"].cpu().numpy(), np.stack(o_stk))
        np.testing.assert_array_equal(state["counters"].cpu().numpy(), np.stack([o_fwd, o_acc], axis=1))
        check_rows(conf_adopted)
    assert all((st != S.TOK_MASKED).all() for st in o_st), "the script should finish the block"
    return chains, o_fwd, o_acc


@pytest.mark.parametrize("L", [32, 64, 5])
def test_blocks_decoded_with_speculative_branches(L):
    chains, fwd, acc = _decode_blocks_both(6, L, 4, seed=100 + L)
    if L >= 32:
        assert {0, 1, 3} <= chains          # the script exercises the chain
    assert (acc == L).all()


def test_plain_threshold_decoding_has_one_branch_and_needs_more_forward_passes():
    _, fwd1, acc1 = _decode_blocks_both(6, 32, 1, seed=7)
    _, fwd4, acc4 = _decode_blocks_both(6, 32, 4, seed=7)
    assert (acc1 == 32).all() and (acc4 == 32).all()
    assert fwd4.sum() < fwd1.sum()          # more tokens per forward pass with the branches (Table 1, TPF)


def test_rows_of_the_glue_feed_the_layer():
    """Two decode steps of 2 sequences x 4 branches x 8 positions: the rows team_seh_step lays out go straight into
    team_moe_forward (device to device), and the layer's result matches the oracle on the oracle's own rows."""
    shape = W.MINI_BF16
    n_seqs, L = 2, shape.block
    import dataclasses
    shape = dataclasses.replace(shape, name="mini_seh", seqs=n_seqs, branches=4)
    weights = W.make_weights(shape)
    layer = P.Layer(shape, weights, 3)
    ocfg = P.oracle_config(shape, 3)
    pred, conf = W.make_decode_script(n_seqs, L, 6, seed=9)
    state, rows = B.seh_alloc(n_seqs, L, 4)
    T = n_seqs * 4 * L
    rng = np.random.default_rng(5)
    y = torch.zeros((T, shape.hidden), dtype=torch.float32, device="cuda")
    try:
        B.team_seh_step(n_seqs, L, 4, TAU, state, None, None, rows)
        for step in range(4):
            x = W.round_to_bf16(rng.standard_normal((T, shape.hidden)).astype(np.float32))
            st = dict(rows)
            out = B.alloc_routing(layer.cfg, T)
            y_before = y.cpu().numpy()
            B.team_moe_forward(layer.ctx, B.to_device(x, B.TEAM_DTYPE_BF16), st, out, y)
            assert B.team_read_status(layer.ctx)[0] == B.TEAM_OK
            h = {n: v.cpu().numpy() for n, v in rows.items()}
            y_ref, ref = O.moe_forward(ocfg, weights, x, h["tok_state"], h["conf"], h["pos"], h["group"], h["branch"],
                                       y_prev=y_before)
            got = B.routing_to_host(out)
            exact, pin = P.compare_routing(ocfg, ref, got, h["group"], f"seh rows step {step}", return_pin=True)
            P.compare_y_rows(shape, ocfg, weights, x, y_ref, ref, got, y.cpu().numpy(), pin, y_before, f"seh rows step {step}",
                             max_unpinned=1)
            B.team_seh_step(n_seqs, L, 4, TAU, state, torch.as_tensor(pred[step]).cuda(), torch.as_tensor(conf[step]).cuda(), rows)
    finally:
        layer.close()
