"""Config 5 at its real depth: 48 SDAR-shaped MoE layers with residual adds, the first decoding block's four
denoising steps, checked layer by layer against the oracle.

The weights (58 GB in bf16) are generated on the device by the seeded generator the benchmark uses; the oracle
gets one layer at a time as a device-to-host copy.  The stack runs on the GPU first (as the benchmark runs it:
one-kernel steps, no dispatch tables), recording for every (step, layer) the activations that entered the layer,
the rows' choices it exported and its output; the check is then teacher-forced -- the oracle is fed the recorded
input of each layer, so a near-tie early in the stack cannot cascade -- and every computed row of every layer is
compared with the oracle at the stated tolerance, the residual add bit for bit."""
import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu


def _round_bf16(a):
    return W.round_to_bf16(np.asarray(a, dtype=np.float32)).astype(np.float64)


@pytest.mark.parametrize("flags,n_layers", [(3, W.C5_LAYERS), (0, 6)], ids=["team_48_layers", "vanilla_6_layers"])
def test_c5_first_block_teacher_forced(flags, n_layers):
    shape = W.C2
    T, H = shape.rows, shape.hidden
    steps = W.make_schedule(shape)
    cfg = P.lib_config(shape, flags)
    ocfg = P.oracle_config(shape, flags)
    dev = torch.device("cuda", 0)
    ctxs, keep = [], []
    try:
        for l in range(n_layers):
            wr, wg, wu, wd = W.device_layer_weights(shape, 5000 + l, dev)
            pk = B.team_pack_w_down(wd)
            del wd
            c = B.team_create(cfg)
            B.team_set_weights(c, wr, wg, wu, pk)
            ctxs.append(c)
            keep.append((wr, wg, wu, pk))
        # ---- the stack on the GPU, everything recorded ----
        y_dev = [torch.full((T, H), 7.0, dtype=torch.float32, device=dev) for _ in range(n_layers)]
        rec = []
        for si, step in enumerate(steps):
            x_dev = B.to_device(step["x"], B.TEAM_DTYPE_BF16, dev)
            st = B.state_to_device(step, dev)
            for l, c in enumerate(ctxs):
                out = {n: v for n, v in B.alloc_routing(cfg, T, dev).items() if n in P.CHOICE_TABLES}
                x_in = x_dev.float().cpu().numpy()
                y_before = y_dev[l].cpu().numpy()
                B.team_moe_forward(c, x_dev, st, out, y_dev[l])
                assert B.team_last_launch_count(c) == 1
                B.team_residual_add(c, x_dev, y_dev[l], T)
                rec.append(dict(si=si, l=l, x_in=x_in, y_before=y_before, y=y_dev[l].cpu().numpy(),
                                x_out=x_dev.float().cpu().numpy(), got=B.routing_to_host(out)))
        for c in ctxs:
            code, detail = B.team_read_status(c)
            assert code == B.TEAM_OK, (code, detail)
        # ---- the check, one layer's weights on the host at a time ----
        n_unpinned = 0
        for l in range(n_layers):
            wr, wg, wu, _ = keep[l]
            _, _, _, wd = W.device_layer_weights(shape, 5000 + l, dev)          # the row-major down projection again
            weights = dict(w_router=wr.cpu().numpy(), w_gate=wg.float().cpu().numpy(), w_up=wu.float().cpu().numpy(),
                           w_down=wd.float().cpu().numpy())
            del wd
            for r in (r for r in rec if r["l"] == l):
                step = steps[r["si"]]
                what = f"c5 stack flags={flags} step={r['si']} layer={l}"
                y_ref, ref = O.moe_forward(ocfg, weights, r["x_in"], step["tok_state"], step["conf"], step["pos"],
                                           step["group"], step["branch"], y_prev=r["y_before"])
                got = r["got"]
                got["n_rows_active"] = int((got["tok_class"] != O.CLS_SKIP).sum())
                exact, pin = P.compare_routing(ocfg, ref, got, step["group"], what, return_pin=True)
                n_unpinned += int((~pin).sum())
                P.compare_y_rows(shape, ocfg, weights, r["x_in"], y_ref, ref, got, r["y"], pin, r["y_before"], what,
                                 max_unpinned=1)        # activations inside the stack are not under a seed's control
                comp = ref["tok_class"] != O.CLS_SKIP
                want = r["x_in"].astype(np.float64).copy()
                want[comp] = _round_bf16(r["x_in"][comp].astype(np.float32) + r["y"][comp])
                np.testing.assert_array_equal(r["x_out"].astype(np.float64), want, err_msg=what)
        # near-ties must stay the exception over the whole block
        assert n_unpinned <= max(2, len(rec) * T // 100)
    finally:
        for c in ctxs:
            B.team_destroy(c)
