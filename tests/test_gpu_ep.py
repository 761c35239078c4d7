"""Expert-parallel sharding on one GPU: the ranks of a 2- and 4-way split are run one after the other as separate
contexts (each with its own experts' weights only), their partial outputs are added on the computed rows, and the
sum is compared with the oracle's full layer output; the routing tables every rank exports are the complete ones.
(No kernel of one rank waits for another, so running them in turn is the same computation.)"""
import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import ep as EP
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu


def _rank_layer(shape, weights, flags, rank, world):
    cfg = P.lib_config(shape, flags, ep_rank=rank, ep_world=world)
    dc = P.dtype_code(shape)
    ctx = B.team_create(cfg)
    E = shape.n_experts
    wg, wu, wd = (B.to_device(weights[n], dc) for n in ("w_gate", "w_up", "w_down"))
    parts = [torch.as_tensor(weights["w_router"]).cuda().contiguous(),
             EP.shard_experts(wg, E, rank, world).contiguous(), EP.shard_experts(wu, E, rank, world).contiguous(),
             EP.shard_experts(B.team_pack_w_down(wd), E, rank, world).contiguous()]
    if shape.dtype == "bf16":
        gu, dt = B.team_pack_w_tiles(wg, wu, wd)
        per = shape.inter * shape.hidden
        parts += [EP.shard_experts(gu, E, rank, world, 2 * per).contiguous(), EP.shard_experts(dt, E, rank, world, per).contiguous()]
    B.team_set_weights(ctx, *parts)
    return ctx, cfg, parts


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("case", ["c2_one_kernel_step", "c2_three_kernels", "c4_b4_streaming", "paper_tensor_memory", "c1_fp32"])
def test_partial_outputs_of_the_ranks_add_up_to_the_layer(case, world):
    shape, tables = {"c2_one_kernel_step": (W.C2, False), "c2_three_kernels": (W.C2, True),
                     "c4_b4_streaming": (W.c4(4), True), "paper_tensor_memory": (W.paper_point(), True),
                     "c1_fp32": (W.C1, True)}[case]
    flags = 3
    weights = W.make_weights(shape)
    ocfg = P.oracle_config(shape, flags)
    steps = W.make_schedule(shape)[1:3]
    ranks = [_rank_layer(shape, weights, flags, r, world) for r in range(world)]
    T, H = shape.rows, shape.hidden
    try:
        y_ref = np.full((T, H), 5.0)
        y_full = torch.full((T, H), 5.0, dtype=torch.float32, device="cuda")
        for si, step in enumerate(steps):
            x_dev = B.to_device(step["x"], P.dtype_code(shape))
            st = B.state_to_device(step)
            y_before = y_full.cpu().numpy()
            partial_sum = torch.zeros_like(y_full)
            gots = []
            for ctx, cfg, _ in ranks:
                out = B.alloc_routing(cfg, T)
                if not tables:
                    out = {n: out[n] for n in P.CHOICE_TABLES}
                y_r = y_full.clone()
                B.team_moe_forward(ctx, x_dev, st, out, y_r)
                assert B.team_read_status(ctx)[0] == B.TEAM_OK
                got = B.routing_to_host(out)
                computed = torch.as_tensor(got["tok_class"] != O.CLS_SKIP).cuda()
                partial_sum += torch.where(computed[:, None], y_r, torch.zeros_like(y_r))
                gots.append(got)
            y_full[computed] = partial_sum[computed]
            y_ref, ref = O.moe_forward(ocfg, weights, step["x"], step["tok_state"], step["conf"], step["pos"],
                                       step["group"], step["branch"], y_prev=y_ref)
            for got in gots:            # every rank routed all rows over all experts
                if "n_rows_active" not in got:
                    got["n_rows_active"] = int((got["tok_class"] != O.CLS_SKIP).sum())
                exact, pin = P.compare_routing(ocfg, ref, got, step["group"], f"{case} world={world} step={si}", return_pin=True)
            P.compare_y_rows(shape, ocfg, weights, step["x"], y_ref, ref, gots[0], y_full.cpu().numpy(), pin, y_before,
                             f"{case} world={world} step={si}")
    finally:
        for ctx, _, _ in ranks:
            B.team_destroy(ctx)


def test_sharding_is_rejected_where_it_cannot_apply():
    import ctypes
    ctx = ctypes.c_void_p()
    bad = B.make_config(2048, 128, 8, 768, ep_rank=0, ep_world=3)          # 128 experts over 3 ranks
    assert B.lib().team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_SHAPE
    bad = B.make_config(2048, 128, 8, 768, n_shared=1, ep_rank=0, ep_world=2)
    assert B.lib().team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_SHAPE
    bad = B.make_config(2048, 128, 8, 768, ep_rank=2, ep_world=2)
    assert B.lib().team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_ARG
