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
        w_down = B.to_device(weights["w_down"], dc)
        self.w = [torch.as_tensor(weights["w_router"]).cuda().contiguous(), B.to_device(weights["w_gate"], dc),
                  B.to_device(weights["w_up"], dc), B.team_pack_w_down(w_down)]
        if shape.dtype == "bf16":        # both layouts: whichever expert kernel the context picks finds its own
            self.w += list(B.team_pack_w_tiles(self.w[1], self.w[2], w_down))
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


PROBS_ATOL = 1e-6      # softmax probabilities: fp32 exp and division against fp64, on the same fp32 logits


def compare_probs(ref, got, what=""):
    """The exported softmax table against the oracle's router: computed rows within PROBS_ATOL, skipped rows zero."""
    comp = ref["tok_class"] != O.CLS_SKIP
    if comp.any():
        np.testing.assert_allclose(got["probs"][comp], ref["probs"][comp], rtol=0, atol=PROBS_ATOL,
                                   err_msg=f"{what} probs")
        np.testing.assert_allclose(got["probs"][comp].sum(axis=1), 1.0, rtol=0, atol=1e-5, err_msg=f"{what} probs sum")
    if (~comp).any():
        assert not got["probs"][~comp].any(), f"{what}: probs of skipped rows must be zero"


def compare_routing(cfg, ref, got, group, what="", return_pin=False):
    """Integer tables bit-exact where pinned; floating-point tables within fp32 rounding."""
    pin, groups_ok = pinned_rows(cfg, ref, group)
    np.testing.assert_array_equal(got["tok_class"], ref["tok_class"], err_msg=what)
    assert got["n_rows_active"] == ref["n_rows_active"], what
    compare_probs(ref, got, what)
    for t in np.flatnonzero(pin):
        np.testing.assert_array_equal(got["topk_idx"][t], ref["topk_idx"][t], err_msg=f"{what} row {t}")
        np.testing.assert_allclose(got["topk_w"][t], ref["topk_w"][t], atol=2e-6, rtol=1e-5, err_msg=what)
        if np.isinf(ref["margin"][t]):
            assert np.isinf(got["margin"][t])
        else:
            assert abs(got["margin"][t] - ref["margin"][t]) < 1e-5
    tables = "perm" in got          # a call may ask for the choices only (no dispatch tables)
    if pin.all() and groups_ok:
        for name in ("group_mask", "expert_count", "expert_offset", "perm", "active") if tables else ("group_mask",):
            np.testing.assert_array_equal(got[name], ref[name], err_msg=f"{what} {name}")
        if tables:
            assert got["n_active"] == ref["n_active"], what
    check_self_consistency(cfg, got, group)
    if return_pin:
        return bool(pin.all() and groups_ok), pin
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
    if "perm" not in got:
        return
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


def y_from_choices(cfg, weights, x, T, row, idx_row, w_row):
    """Layer output of one row from a given set of choices: sum_j w_j * expert(idx_j)(x) + shared experts.
    Used for rows whose own choice is not pinned (a near-tie): the oracle's expert arithmetic on the choice the
    library reports, so that the row's y is still checked against the oracle and never against itself."""
    y = np.zeros(cfg.hidden, dtype=np.float64)
    xr = np.asarray(x)[row:row + 1]
    for e, wt in zip(idx_row, w_row):
        y += float(wt) * O.expert_ffn(xr, weights["w_gate"][int(e)], weights["w_up"][int(e)], weights["w_down"][int(e)])[0]
    for sh in range(cfg.n_shared):
        e = cfg.n_experts + sh
        y += O.expert_ffn(xr, weights["w_gate"][e], weights["w_up"][e], weights["w_down"][e])[0]
    return y


MIN_PINNED_FRACTION = 0.99     # of the rows of a step; below it the seed is a bad one and the test must say so


def compare_y_rows(shape, cfg, weights, x, ref_y, ref, got, got_y, pin, y_before, what="", max_unpinned=None):
    """Every computed row against the oracle at the stated tolerance: pinned rows against the oracle's layer
    output, the others against the oracle's expert arithmetic on the choices the library reports.  Skipped rows
    must be bit-identical to what was there before.  Returns (max relative error, oracle y with the unpinned rows
    replaced).  max_unpinned: how many rows of the step may have a near-tie (default: 1 % of the rows, i.e. none in
    a small step; callers whose inputs are not under a seed's control, such as the activations inside a stack, say
    how many they tolerate)."""
    tol = TOL_BF16 if shape.dtype == "bf16" else TOL_F32
    cls = ref["tok_class"]
    T = len(cls)
    comp = cls != O.CLS_SKIP
    n_unpinned = int((~pin).sum())
    if max_unpinned is None:
        max_unpinned = int((1.0 - MIN_PINNED_FRACTION) * T)
    assert n_unpinned <= max_unpinned, \
        f"{what}: {n_unpinned} of {T} rows have a near-tie: too many for a meaningful comparison, pick another seed"
    want = np.array(ref_y, dtype=np.float64)
    for t in np.flatnonzero(comp & ~pin):
        want[t] = y_from_choices(cfg, weights, x, T, t, got["topk_idx"][t], got["topk_w"][t])
    rel = 0.0
    if comp.any():
        scale = np.abs(want[comp]).max()
        err_rows = np.abs(got_y[comp] - want[comp]).max(axis=1)
        worst = int(np.flatnonzero(comp)[err_rows.argmax()])
        assert err_rows.max() <= tol * scale, \
            f"{what}: row {worst} max|err| {err_rows.max():.3e} > {tol} * {scale:.3e}"
        rel = float(err_rows.max() / scale) if scale > 0 else 0.0
    if (~comp).any():
        np.testing.assert_array_equal(got_y[~comp], y_before[~comp], err_msg=f"{what}: cached rows changed")
    return rel, want


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


CHOICE_TABLES = ("probs", "topk_idx", "topk_w", "margin", "tok_class", "group_mask")


def run_schedule(shape, weights, steps, flags, force_simt=False, policy_switch=None, tables=True, knobs=(), **kw):
    """Runs every step of a schedule through team_moe_forward and the oracle; returns per-step stats.

    Every computed row of every step is compared with the oracle (compare_y_rows): there is no step whose layer
    output goes unchecked.  `policy_switch` = (step index, dict of policy fields): from that step on both sides use
    the changed policy (the library through team_set_policy on the same context)."""
    ocfg = oracle_config(shape, flags, **kw)
    layer = Layer(shape, weights, flags, **kw)
    if force_simt:
        B.team_debug_force_simt(layer.ctx, 1)
    for knob, value in knobs:
        B.team_debug_knob(layer.ctx, knob, value)
    T = steps[0]["x"].shape[0]
    y_dev = torch.full((T, shape.hidden), 123.0, dtype=torch.float32, device="cuda")
    y_ref = np.full((T, shape.hidden), 123.0)
    stats = []
    try:
        for si, step in enumerate(steps):
            if policy_switch is not None and si == policy_switch[0]:
                import dataclasses
                changed = dict(policy_switch[1])
                new_flags = changed.pop("flags", flags)
                ocfg = dataclasses.replace(ocfg, flags=new_flags, **changed)
                for name, v in changed.items():
                    setattr(layer.cfg, name, v)
                layer.cfg.flags = new_flags
                B.team_set_policy(layer.ctx, layer.cfg)
            x_dev = B.to_device(step["x"], dtype_code(shape))
            st = B.state_to_device(step)
            st["step_index"] = si
            out = B.alloc_routing(layer.cfg, T)
            if not tables:
                out = {n: out[n] for n in CHOICE_TABLES}
            y_before = y_dev.cpu().numpy()
            B.team_moe_forward(layer.ctx, x_dev, st, out, y_dev)
            code, detail = B.team_read_status(layer.ctx)
            assert code == B.TEAM_OK, f"device status {code} detail {detail}"
            got = B.routing_to_host(out)
            if not tables:
                comp = got["tok_class"] != O.CLS_SKIP
                got["n_rows_active"] = int(comp.sum())
                chosen = set(got["topk_idx"][comp].ravel().tolist())
                got["n_active"] = len(chosen) + (shape.n_shared if comp.any() else 0)
            y_ref, ref = O.moe_forward(ocfg, weights, step["x"], step["tok_state"], step["conf"], step["pos"],
                                       step["group"], step["branch"], y_prev=y_ref, step_index=si)
            what = f"{shape.name} flags={ocfg.flags} step={si}"
            exact, pin = compare_routing(ocfg, ref, got, step["group"], what, return_pin=True)
            got_y = y_dev.cpu().numpy()
            rel, y_ref = compare_y_rows(shape, ocfg, weights, step["x"], y_ref, ref, got, got_y, pin, y_before, what)
            stats.append(dict(step=si, n_active=got["n_active"], rows=got["n_rows_active"], rel_err=rel,
                              exact=exact, pinned=int(pin.sum()), classes=ref["tok_class"].copy(),
                              launches=B.team_last_launch_count(layer.ctx)))
    finally:
        layer.close()
    return stats
