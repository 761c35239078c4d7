"""GPU parity of the attention half of delayed caching (team_block_attention) against the oracle: a block decoded
over several steps with its in-block KV cache carried from step to step on both sides -- outputs of the computed
rows within tolerance, untouched rows bit-identical, the cache after every pass bit for bit."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as A
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W

pytestmark = pytest.mark.gpu
TOL = 1e-4          # max |err| <= TOL * ||out||_inf: bf16 inputs are exact on both sides, the kernel accumulates in fp32


def _bf16(rng, *shape):
    return W.round_to_bf16(rng.standard_normal(shape).astype(np.float32))


def _dev(a):
    return torch.as_tensor(a).cuda().to(torch.bfloat16).contiguous()


@pytest.mark.parametrize("flags", [0, B.TEAM_F_DCD], ids=["recompute_all", "delayed_caching"])
@pytest.mark.parametrize("shape", [W.C2, W.paper_point(), W.c4(4)], ids=lambda s: s.name)
@pytest.mark.parametrize("d,Hq,Hkv,P", [(128, 8, 2, 70), (64, 4, 4, 33)], ids=["d128_gqa4", "d64_mha"])
def test_block_attention_over_a_schedule(shape, flags, d, Hq, Hkv, P):
    rng = np.random.default_rng(shape.seed + d)
    steps = W.make_schedule(shape)[:4]                    # token states, positions, groups, branches of the layer's schedule
    S, Bn, L, T = shape.seqs, shape.branches, shape.block, shape.rows
    cfg = B.team_attn_config(Hq, Hkv, d, L, S, Bn, P, flags)
    kp, vp = _bf16(rng, S, P, Hkv, d), _bf16(rng, S, P, Hkv, d)
    plen = rng.integers(P // 2, P + 1, S).astype(np.int32)
    plen[0] = P
    kb, vb = np.zeros((S, L, Hkv, d), np.float32), np.zeros((S, L, Hkv, d), np.float32)
    kb_dev, vb_dev = _dev(kb), _dev(vb)
    out_dev = torch.full((T, Hq, d), 3.0, dtype=torch.float32, device="cuda")
    out_ref = np.full((T, Hq, d), 3.0)
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    for si, step in enumerate(steps):
        q, k, v = _bf16(rng, T, Hq, d), _bf16(rng, T, Hkv, d), _bf16(rng, T, Hkv, d)
        st = B.state_to_device(step)
        before = out_dev.cpu().numpy()
        rc = B.team_block_attention(cfg, st, _dev(q), _dev(k), _dev(v), _dev(kp), _dev(vp), torch.as_tensor(plen).cuda(),
                                    kb_dev, vb_dev, out_dev, status)
        assert rc == B.TEAM_OK
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0, 0]
        out_ref, kb, vb = A.block_attention(q, k, v, kp, vp, plen, kb, vb, step["tok_state"], step["pos"], step["group"],
                                            step["branch"], L, flags, out_prev=out_ref)
        got = out_dev.cpu().numpy()
        comp = A.computed_rows(step["tok_state"], flags)
        assert comp.any()
        err = np.abs(got[comp] - out_ref[comp]).max()
        assert err <= TOL * np.abs(out_ref[comp]).max(), f"step {si}: {err}"
        np.testing.assert_array_equal(got[~comp], before[~comp])                     # cached tokens: no query, no output
        out_ref[~comp] = got[~comp]
        np.testing.assert_array_equal(kb_dev.float().cpu().numpy(), kb.astype(np.float32))   # the cache after insertion
        np.testing.assert_array_equal(vb_dev.float().cpu().numpy(), vb.astype(np.float32))
    if flags:
        assert (kb != 0).any()          # something was inserted along the way


@pytest.mark.parametrize("flags", [0, B.TEAM_F_DCD], ids=["recompute_all", "delayed_caching"])
@pytest.mark.parametrize("d,Hq,Hkv", [(128, 16, 2), (64, 8, 1)], ids=["d128", "d64"])
def test_block_attention_long_prefix(flags, d, Hq, Hkv):
    """A prefix of many key tiles with a ragged end, eight query heads per key/value head (more (row, head) pairs than
    one CTA holds) and few enough CTAs that the keys are split over a cluster; queries scaled up so that the running
    maximum keeps moving (the rescaling of the output accumulator is exercised, not only its first tile)."""
    shape = W.paper_point()
    rng = np.random.default_rng(977 + d)
    steps = W.make_schedule(shape)[:2]
    S, Bn, L, T = shape.seqs, shape.branches, shape.block, shape.rows
    P = 1000
    cfg = B.team_attn_config(Hq, Hkv, d, L, S, Bn, P, flags)
    kp, vp = _bf16(rng, S, P, Hkv, d), _bf16(rng, S, P, Hkv, d)
    plen = np.full(S, 937, np.int32)
    kb, vb = _bf16(rng, S, L, Hkv, d), _bf16(rng, S, L, Hkv, d)
    kb_dev, vb_dev = _dev(kb), _dev(vb)
    out_dev = torch.full((T, Hq, d), 3.0, dtype=torch.float32, device="cuda")
    out_ref = np.full((T, Hq, d), 3.0)
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    for si, step in enumerate(steps):
        q = W.round_to_bf16((6.0 * rng.standard_normal((T, Hq, d))).astype(np.float32))
        k, v = _bf16(rng, T, Hkv, d), _bf16(rng, T, Hkv, d)
        rc = B.team_block_attention(cfg, B.state_to_device(step), _dev(q), _dev(k), _dev(v), _dev(kp), _dev(vp),
                                    torch.as_tensor(plen).cuda(), kb_dev, vb_dev, out_dev, status)
        assert rc == B.TEAM_OK
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0, 0]
        out_ref, kb, vb = A.block_attention(q, k, v, kp, vp, plen, kb, vb, step["tok_state"], step["pos"], step["group"],
                                            step["branch"], L, flags, out_prev=out_ref)
        got = out_dev.cpu().numpy()
        comp = A.computed_rows(step["tok_state"], flags)
        err = np.abs(got[comp] - out_ref[comp]).max()
        assert err <= TOL * np.abs(out_ref[comp]).max(), f"step {si}: {err}"
        out_ref[~comp] = got[~comp]
        np.testing.assert_array_equal(kb_dev.float().cpu().numpy(), kb.astype(np.float32))
        np.testing.assert_array_equal(vb_dev.float().cpu().numpy(), vb.astype(np.float32))


def test_block_attention_rejects_what_it_cannot_run():
    z = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    st = dict(tok_state=torch.zeros(4, dtype=torch.uint8, device="cuda"), pos=torch.arange(4, dtype=torch.int32, device="cuda"),
              group=torch.zeros(4, dtype=torch.int32, device="cuda"), branch=torch.zeros(4, dtype=torch.int32, device="cuda"))
    out = torch.zeros(16, dtype=torch.float32, device="cuda")
    plen = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad_dim = B.team_attn_config(2, 2, 96, 4, 1, 1, 0, 0)
    assert B.team_block_attention(bad_dim, st, z, z, z, z, z, plen, z, z, out) == B.TEAM_ERR_SHAPE
    bad_heads = B.team_attn_config(3, 2, 64, 4, 1, 1, 0, 0)
    assert B.team_block_attention(bad_heads, st, z, z, z, z, z, plen, z, z, out) == B.TEAM_ERR_SHAPE
    bad_rows = B.team_attn_config(2, 2, 64, 8, 1, 1, 0, 0)               # 8 rows expected, 4 given
    assert B.team_block_attention(bad_rows, st, z, z, z, z, z, plen, z, z, out) == B.TEAM_ERR_ARG


def test_block_attention_reports_a_broken_row_layout():
    """Rows of a run out of position order: the layout contract is checked on the device and reported, nothing faults."""
    L, d = 4, 64
    cfg = B.team_attn_config(2, 2, d, L, 1, 1, 4, 0)
    rng = np.random.default_rng(0)
    st = dict(tok_state=torch.zeros(L, dtype=torch.uint8, device="cuda"),
              pos=torch.tensor([0, 2, 1, 3], dtype=torch.int32, device="cuda"),
              group=torch.zeros(L, dtype=torch.int32, device="cuda"), branch=torch.zeros(L, dtype=torch.int32, device="cuda"))
    q, k, v = _dev(_bf16(rng, L, 2, d)), _dev(_bf16(rng, L, 2, d)), _dev(_bf16(rng, L, 2, d))
    kp = _dev(_bf16(rng, 1, 4, 2, d))
    kb = _dev(np.zeros((1, L, 2, d), np.float32))
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    out = torch.zeros((L, 2, d), dtype=torch.float32, device="cuda")
    assert B.team_block_attention(cfg, st, q, k, v, kp, kp.clone(), torch.tensor([4], dtype=torch.int32, device="cuda"),
                                  kb, kb.clone(), out, status) == B.TEAM_OK
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [B.TEAM_ERR_STATE, 40]
