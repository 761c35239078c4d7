"""Helpers shared by the GPU parity tests: run the CUDA library and the oracle on the same seeded
inputs and compare them element by element."""
import numpy as np
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B

MARGIN = 1e-5          # integer results are compared where every ordering decision is clearer than this
TOL_BF16 = 2e-2        # max |err| <= TOL * ||y||_inf   (bf16 weights)
TOL_F32 = 1e-4         # same form for the fp32 configuration


def dtype_code(shape):
    return B.TEAM_DTYPE_BF16 if shape.dtype == "bf16" else B.TEAM_DTYPE_F32


def oracle_config(shape, flags, **kw):
    return O.Config(hidden=shape.hidden, n_experts=shape.n_experts, top_k=shape.top_k, inter=shape.inter,
                    n_shared=shape.n_shared, flags=flags, tau_hot=shape.tau_hot, L_hot=shape.L_hot,
                    max_groups=shape.seqs, **kw)


def lib_config(shape, flags, max_rows=None, **kw):
    return B.make_config(shape.hidden, shape.n_experts, shape.top_k, shape.inter, shape.n_shared,
                         max_rows=max_rows or shape.rows, max_groups=shape.seqs, dtype=dtype_code(shape),
                         flags=flags, tau_hot=shape.tau_hot, L_hot=shape.L_hot, **kw)


class Layer:
    """A context with its weights on the device."""

    def __init__(self, shape, weights, flags, **kw):
        self.shape, self.cfg = shape, lib_config(shape, flags, **kw)
        self.ctx = B.team_create(self.cfg)
        dc = dtype_code(shape)
        self.w = [torch.as_tensor(weights["w_router"]).cuda().contiguous(), B.to_device(weights["w_gate"], dc),
                  B.to_device(weights["w_up"], dc), B.team_pack_w_down(B.to_device(weights["w_down"], dc))]
        B.team_set_weights(self.ctx, *self.w)

    def close(self):
        B.team_destroy(self.ctx)


def ordering_margin(logits32_row, idx_row, candidates):
    """Smallest logit gap among the ordering decisions behind a row's top-k (incl. the cut-off)."""
    l = logits32_row.astype(np.float64)
    order = sorted(candidates, key=lambda e: (-l[e], e))
    k = len(idx_row)
    top = order[:k + 1]
    gaps = [l[top[j]] - l[top[j + 1]] for j in range(len(top) - 1)]
    return min(gaps) if gaps else np.inf


def pinned_rows(cfg, ref, group):
    """Rows whose integer results must match bit for bit (cascade through E_A included)."""
    T, E = ref["logits"].shape
    cls = ref["tok_class"]
    own = np.zeros(T, dtype=bool)
    for t in range(T):
        if cls[t] == O.CLS_SKIP:
            own[t] = True
            continue
        if cls[t] == O.CLS_FIRST:
            cand = range(E)
        else:
            gm = ref["group_mask"][group[t]]
            cand = [e for e in range(E) if (int(gm[e // 64]) >> (e % 64)) & 1]
        own[t] = ordering_margin(ref["logits"][t], ref["topk_idx"][t], cand) > MARGIN
    group_ok = {}
    for t in range(T):
        if cls[t] == O.CLS_FIRST:
            group_ok[group[t]] = group_ok.get(group[t], True) and own[t]
    return np.array([own[t] and (cls[t] != O.CLS_COLD or group_ok.get(group[t], True)) for t in range(T)]), \
        all(group_ok.values())


def compare_routing(cfg, ref, got, group, what=""):
    """Integer tables bit-exact where pinned; floating-point tables within fp32 rounding."""
    pin, groups_ok = pinned_rows(cfg, ref, group)
    np.testing.assert_array_equal(got["tok_class"], ref["tok_class"], err_msg=what)
    assert got["n_rows_active"] == ref["n_rows_active"], what
    for t in np.flatnonzero(pin):
        np.testing.assert_array_equal(got["topk_idx"][t], ref["topk_idx"][t], err_msg=f"{what} row {t}")
        np.testing.assert_allclose(got["topk_w"][t], ref["topk_w"][t], atol=2e-6, rtol=1e-5, err_msg=what)
        if np.isinf(ref["margin"][t]):
            assert np.isinf(got["margin"][t])
        else:
            assert abs(got["margin"][t] - ref["margin"][t]) < 1e-5
    if pin.all() and groups_ok:
        for name in ("group_mask", "expert_count", "expert_offset", "perm", "active"):
            np.testing.assert_array_equal(got[name], ref[name], err_msg=f"{what} {name}")
        assert got["n_active"] == ref["n_active"], what
    check_self_consistency(cfg, got, group)
    return bool(pin.all() and groups_ok)


def check_self_consistency(cfg, got, group):
    """Properties that hold for any valid answer, whatever near-ties decided."""
    T, k = got["topk_idx"].shape
    E, ns = cfg.n_experts, cfg.n_shared
    cls = got["tok_class"]
    union = {}
    for t in range(T):
        if cls[t] == O.CLS_FIRST:
            union.setdefault(group[t], set()).update(got["topk_idx"][t].tolist())
    for g, s in union.items():
        bits = {e for e in range(E) if (int(got["group_mask"][g, e // 64]) >> (e % 64)) & 1}
        assert bits == s
    for t in range(T):
        if cls[t] == O.CLS_COLD:
            assert set(got["topk_idx"][t].tolist()) <= union[group[t]]
        if cls[t] != O.CLS_SKIP:
            assert len(set(got["topk_idx"][t].tolist())) == k
            assert abs(got["topk_w"][t].sum() - 1.0) < 1e-5 or not cfg.norm_topk
    rows = [t for t in range(T) if cls[t] != O.CLS_SKIP]
    S = len(rows) * (k + ns)
    cnt = got["expert_count"]
    assert cnt.sum() == S and got["expert_offset"][-1] == S
    np.testing.assert_array_equal(np.diff(got["expert_offset"]), cnt)
    perm = got["perm"][:S]
    assert len(set(perm.tolist())) == S and np.all(got["perm"][S:] == -1)
    for e in range(E + ns):
        seg = perm[got["expert_offset"][e]:got["expert_offset"][e + 1]]
        assert np.all(np.diff(seg) > 0)
        for sid in seg:
            if sid < T * k:
                assert got["topk_idx"][sid // k, sid % k] == e
            else:
                assert e == E + (sid - T * k) // T and (sid - T * k) % T in rows
    np.testing.assert_array_equal(got["active"], np.flatnonzero(cnt > 0))


def compare_y(shape, ref_y, got_y, cls, y_before, what=""):
    tol = TOL_BF16 if shape.dtype == "bf16" else TOL_F32
    comp = cls != O.CLS_SKIP
    if comp.any():
        scale = np.abs(ref_y[comp]).max()
        err = np.abs(got_y[comp] - ref_y[comp]).max()
        assert err <= tol * scale, f"{what}: max|err| {err:.3e} > {tol} * {scale:.3e}"
    if (~comp).any():
        np.testing.assert_array_equal(got_y[~comp], y_before[~comp], err_msg=f"{what}: cached rows changed")
    return (np.abs(got_y[comp] - ref_y[comp]).max() / np.abs(ref_y[comp]).max()) if comp.any() else 0.0


def run_schedule(shape, weights, steps, flags, force_simt=False, check_routing=True, **kw):
    """Runs every step of a schedule through team_moe_forward and the oracle; returns per-step stats."""
    ocfg = oracle_config(shape, flags, **kw)
    layer = Layer(shape, weights, flags, **kw)
    if force_simt:
        B.team_debug_force_simt(layer.ctx, 1)
    T = steps[0]["x"].shape[0]
    y_dev = torch.full((T, shape.hidden), 123.0, dtype=torch.float32, device="cuda")
    y_ref = np.full((T, shape.hidden), 123.0)
    stats = []
    try:
        for si, step in enumerate(steps):
            x_dev = B.to_device(step["x"], dtype_code(shape))
            st = B.state_to_device(step)
            out = B.alloc_routing(layer.cfg, T)
            y_before = y_dev.cpu().numpy()
            B.team_moe_forward(layer.ctx, x_dev, st, out, y_dev)
            code, detail = B.team_read_status(layer.ctx)
            assert code == B.TEAM_OK, f"device status {code} detail {detail}"
            got = B.routing_to_host(out)
            y_ref, ref = O.moe_forward(ocfg, weights, step["x"], step["tok_state"], step["conf"], step["pos"],
                                       step["group"], step["branch"], y_prev=y_ref)
            what = f"{shape.name} flags={flags} step={si}"
            exact = compare_routing(ocfg, ref, got, step["group"], what) if check_routing else True
            got_y = y_dev.cpu().numpy()
            if exact:
                rel = compare_y(shape, y_ref, got_y, ref["tok_class"], y_before, what)
            else:
                rel = float("nan")      # a near-tie changed an expert choice; y is checked by self-consistency only
                y_ref = got_y.astype(np.float64)
            stats.append(dict(step=si, n_active=got["n_active"], rows=got["n_rows_active"], rel_err=rel,
                              exact=exact, launches=B.team_last_launch_count(layer.ctx)))
    finally:
        layer.close()
    return stats
