"""Pins for the oracle's expert FFN, weighted combine, delayed caching and stack glue."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import team_oracle as O


def _weights(rng, E, H, I, ns=0, std=0.3):
    return dict(w_router=(std * rng.standard_normal((E, H))).astype(np.float32),
                w_gate=(std * rng.standard_normal((E + ns, I, H))).astype(np.float32),
                w_up=(std * rng.standard_normal((E + ns, I, H))).astype(np.float32),
                w_down=(std * rng.standard_normal((E + ns, H, I))).astype(np.float32))


def _torch_mlp(x, wg, wu, wd):
    x, wg, wu, wd = (torch.from_numpy(np.asarray(a, dtype=np.float64)) for a in (x, wg, wu, wd))
    return F.linear(F.silu(F.linear(x, wg)) * F.linear(x, wu), wd).numpy()


def _state(T, kind="masked"):
    st = np.zeros(T, dtype=np.uint8)
    return st, np.full(T, 0.1, np.float32), np.arange(T), np.zeros(T, int), np.zeros(T, int)


def check_ffn_against_plain_loops(O):
    rng = np.random.default_rng(1)
    H, I = 5, 3
    x = rng.standard_normal((2, H))
    wg, wu, wd = rng.standard_normal((I, H)), rng.standard_normal((I, H)), rng.standard_normal((H, I))
    out = O.expert_ffn(x, wg, wu, wd)
    for t in range(2):
        a = []
        for i in range(I):
            g = sum(wg[i, h] * x[t, h] for h in range(H))
            u = sum(wu[i, h] * x[t, h] for h in range(H))
            a.append(g / (1.0 + math.exp(-g)) * u)
        for h in range(H):
            assert out[t, h] == pytest.approx(sum(wd[h, i] * a[i] for i in range(I)), rel=1e-12)


def check_ffn_against_library_ops(O):
    rng = np.random.default_rng(2)
    x = rng.standard_normal((4, 16))
    wg, wu, wd = rng.standard_normal((12, 16)), rng.standard_normal((12, 16)), rng.standard_normal((16, 12))
    np.testing.assert_allclose(O.expert_ffn(x, wg, wu, wd), _torch_mlp(x, wg, wu, wd), rtol=1e-12, atol=1e-12)


def check_single_expert_layer_is_a_dense_mlp(O):
    rng = np.random.default_rng(3)
    T, H, I = 6, 16, 8
    w = _weights(rng, 1, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    cfg = O.Config(hidden=H, n_experts=1, top_k=1, inter=I, flags=0)
    y, r = O.moe_forward(cfg, w, x, *_state(T))
    np.testing.assert_allclose(y, _torch_mlp(x, w["w_gate"][0], w["w_up"][0], w["w_down"][0]),
                               rtol=1e-12, atol=1e-13)
    assert r["n_active"] == 1


def check_full_k_is_the_softmax_mixture(O):
    rng = np.random.default_rng(4)
    T, E, H, I = 5, 4, 12, 6
    w = _weights(rng, E, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    cfg = O.Config(hidden=H, n_experts=E, top_k=E, inter=I, flags=0)
    y, _ = O.moe_forward(cfg, w, x, *_state(T))
    logits = torch.from_numpy(x.astype(np.float64)) @ torch.from_numpy(w["w_router"].astype(np.float64)).T
    p = torch.softmax(logits.float().double(), dim=1).numpy()
    ref = sum(p[:, e:e + 1] * _torch_mlp(x, w["w_gate"][e], w["w_up"][e], w["w_down"][e]) for e in range(E))
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-13)


def check_topk_mixture_against_library_topk(O):
    rng = np.random.default_rng(5)
    T, E, k, H, I = 7, 8, 3, 10, 4
    w = _weights(rng, E, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    cfg = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=0)
    y, _ = O.moe_forward(cfg, w, x, *_state(T))
    logits = (torch.from_numpy(x.astype(np.float64)) @ torch.from_numpy(w["w_router"].astype(np.float64)).T).float()
    p = torch.softmax(logits.double(), dim=1)
    val, idx = torch.topk(p, k, dim=1)
    val = (val / val.sum(dim=1, keepdim=True)).numpy()
    ref = np.zeros((T, H))
    for t in range(T):
        for j in range(k):
            e = int(idx[t, j])
            ref[t] += val[t, j] * _torch_mlp(x[t:t + 1], w["w_gate"][e], w["w_up"][e], w["w_down"][e])[0]
    np.testing.assert_allclose(y, ref, rtol=1e-11, atol=1e-13)


def check_zero_down_and_linearity(O):
    rng = np.random.default_rng(6)
    T, E, k, H, I = 4, 6, 2, 8, 4
    w = _weights(rng, E, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    cfg = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=0)
    y, _ = O.moe_forward(cfg, w, x, *_state(T))
    w0 = dict(w, w_down=np.zeros_like(w["w_down"]))
    assert np.all(O.moe_forward(cfg, w0, x, *_state(T))[0] == 0)
    w2 = dict(w, w_down=2 * w["w_down"])
    np.testing.assert_allclose(O.moe_forward(cfg, w2, x, *_state(T))[0], 2 * y, rtol=1e-13)


def check_shared_expert_adds_a_dense_mlp(O):
    rng = np.random.default_rng(7)
    T, E, k, H, I = 5, 6, 2, 8, 4
    w = _weights(rng, E, H, I, ns=1)
    x = rng.standard_normal((T, H)).astype(np.float32)
    cfg1 = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, n_shared=1, flags=0)
    cfg0 = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, n_shared=0, flags=0)
    y1, r1 = O.moe_forward(cfg1, w, x, *_state(T))
    y0, _ = O.moe_forward(cfg0, w, x, *_state(T))
    np.testing.assert_allclose(y1 - y0, _torch_mlp(x, w["w_gate"][E], w["w_up"][E], w["w_down"][E]),
                               rtol=1e-10, atol=1e-12)
    assert r1["active"][-1] == E and r1["expert_count"][E] == T


def check_cached_rows_keep_previous_output(O):
    rng = np.random.default_rng(8)
    T, E, k, H, I = 6, 8, 2, 8, 4
    w = _weights(rng, E, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    st = np.array([O.TOK_CACHED, O.TOK_CACHED, O.TOK_NEW, O.TOK_MASKED, O.TOK_MASKED, O.TOK_MASKED], np.uint8)
    _, conf, pos, grp, br = _state(T)
    y_prev = rng.standard_normal((T, H))
    cfg = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=O.F_DCD | O.F_LAC, L_hot=1, prefix_decoded=0)
    y, r = O.moe_forward(cfg, w, x, st, conf, pos, grp, br, y_prev=y_prev)
    np.testing.assert_array_equal(y[:2], y_prev[:2])
    assert r["n_rows_active"] == 4
    # computed rows equal what the vanilla layer gives them when their expert choice is the same
    van = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=0)
    yv, rv = O.moe_forward(van, w, x, st, conf, pos, grp, br)
    for t in range(2, T):
        if set(r["topk_idx"][t]) == set(rv["topk_idx"][t]):
            np.testing.assert_allclose(y[t], yv[t], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(y[2], yv[2], rtol=1e-12, atol=1e-14)   # the NEW row always routes freely


PINS = [check_ffn_against_plain_loops, check_ffn_against_library_ops,
        check_single_expert_layer_is_a_dense_mlp, check_full_k_is_the_softmax_mixture,
        check_topk_mixture_against_library_topk, check_zero_down_and_linearity,
        check_shared_expert_adds_a_dense_mlp, check_cached_rows_keep_previous_output]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(O)


def test_stack_glue_is_a_residual_add_on_computed_rows():
    rng = np.random.default_rng(9)
    T, E, k, H, I = 4, 6, 2, 8, 4
    layers = [_weights(rng, E, H, I) for _ in range(3)]
    x = rng.standard_normal((T, H)).astype(np.float32)
    st = np.array([O.TOK_CACHED, O.TOK_NEW, O.TOK_MASKED, O.TOK_MASKED], np.uint8)
    _, conf, pos, grp, br = _state(T)
    cfg = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=O.F_DCD, L_hot=1)
    out, n_act = O.stack_forward(cfg, layers, x, st, conf, pos, grp, br)
    ref = x.astype(np.float64).copy()
    for w in layers:
        y, _ = O.moe_forward(cfg, w, ref, st, conf, pos, grp, br)
        ref[1:] = ref[1:] + y[1:]
    np.testing.assert_allclose(out, ref, rtol=1e-13)
    np.testing.assert_array_equal(out[0], x[0].astype(np.float64))
    assert len(n_act) == 3


def test_stack_with_single_expert_layers_is_a_residual_mlp_stack_with_rounding():
    """Pin of the stack glue against library ops, including the store-back rounding: with one expert and k = 1 every
    layer is a dense SwiGLU MLP, so the stack is x <- round(x + mlp_l(x)) layer after layer, written here with torch
    CPU ops and a bf16 round trip through torch's own conversion."""
    rng = np.random.default_rng(10)
    T, H, I, L = 5, 16, 8, 4
    layers = [_weights(rng, 1, H, I) for _ in range(L)]
    x = torch.from_numpy(rng.standard_normal((T, H)).astype(np.float32)).to(torch.bfloat16).float().numpy()
    cfg = O.Config(hidden=H, n_experts=1, top_k=1, inter=I, flags=0)

    def to_bf16(a):
        return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).double().numpy()

    for round_fn in (None, to_bf16):
        out, n_act = O.stack_forward(cfg, layers, x, *_state(T), round_fn=round_fn)
        ref = x.astype(np.float64)
        for w in layers:
            ref = ref + _torch_mlp(ref, w["w_gate"][0], w["w_up"][0], w["w_down"][0])
            if round_fn is not None:
                ref = to_bf16(ref)
        np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
        assert n_act == [1] * L
    # zero down projections: the stack is the identity
    for w in layers:
        w["w_down"][:] = 0
    out, _ = O.stack_forward(cfg, layers, x, *_state(T), round_fn=to_bf16)
    np.testing.assert_array_equal(out, x.astype(np.float64))


def test_periodic_refresh_recomputes_everything_every_nth_step():
    """Sec. 4.1 (second paragraph) / Table 3: Refresh-N recomputes all tokens every N steps.  Pins: the computed-row
    counts over an 8-step schedule follow by hand; a refresh step equals the same step with delayed caching off
    (cached tokens are first-round rows there too); every other step equals plain delayed caching."""
    rng = np.random.default_rng(12)
    T, E, k, H, I = 4, 6, 2, 8, 4
    w = _weights(rng, E, H, I)
    x = rng.standard_normal((T, H)).astype(np.float32)
    _, conf, pos, grp, br = _state(T)
    # tokens 0..3 are accepted after steps 0, 2, 4, 6: NEW on the next step, cached from the one after
    sched = []
    for s in range(8):
        st = np.zeros(T, np.uint8)
        for p in range(T):
            if s == 2 * p + 1:
                st[p] = O.TOK_NEW
            elif s > 2 * p + 1:
                st[p] = O.TOK_CACHED
        sched.append(st)
    want = {0: [4, 4, 3, 3, 2, 2, 1, 1], 4: [4, 4, 3, 3, 4, 2, 1, 1], 8: [4, 4, 3, 3, 2, 2, 1, 1], 2: [4, 4, 4, 3, 4, 2, 4, 1]}
    for n, rows in want.items():
        cfg = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=O.F_DCD | O.F_LAC, L_hot=1, refresh_every=n)
        plain = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=O.F_DCD | O.F_LAC, L_hot=1)
        nodcd = O.Config(hidden=H, n_experts=E, top_k=k, inter=I, flags=O.F_LAC, L_hot=1)
        got = []
        for s, st in enumerate(sched):
            y, r = O.moe_forward(cfg, w, x, st, conf, pos, grp, br, step_index=s)
            got.append(r["n_rows_active"])
            same_as = nodcd if (n > 0 and s % n == 0) else plain
            y2, r2 = O.moe_forward(same_as, w, x, st, conf, pos, grp, br)
            np.testing.assert_array_equal(y, y2)
            np.testing.assert_array_equal(r["tok_class"], r2["tok_class"])
        assert got == rows, (n, got)


# --- planted mistakes: each must be caught by at least one pin ---------------------
def _fails(pins, mod):
    for pin in pins:
        try:
            pin(mod)
        except AssertionError:
            return True
    return False


class _Mutant:
    """The oracle module with one function replaced."""

    def __init__(self, **repl):
        self.__dict__.update({k: getattr(O, k) for k in dir(O) if not k.startswith("__")})
        self.__dict__.update(repl)
        # module-level functions look names up in O's globals, so rebuild the callers
        import types
        g = dict(O.__dict__)
        g.update(repl)
        for name in ("moe_forward", "select_experts", "stack_forward"):
            if name not in repl:
                f = getattr(O, name)
                self.__dict__[name] = types.FunctionType(f.__code__, g, name, f.__defaults__)
                g[name] = self.__dict__[name]


def _swap_gate_up(x, wg, wu, wd):
    return O.expert_ffn(x, wu, wg, wd)


def _no_sigmoid_scale(x, wg, wu, wd):
    x64 = np.asarray(x, np.float64)
    g = x64 @ np.asarray(wg, np.float64).T
    u = x64 @ np.asarray(wu, np.float64).T
    return (1.0 / (1.0 + np.exp(-g)) * u) @ np.asarray(wd, np.float64).T


def _transposed_down(x, wg, wu, wd):
    """The down projection read with its two axes exchanged: the [H, I] matrix is taken as if it were stored [I, H]
    (same bytes, other strides), which is what a transposed operand is for a non-square matrix."""
    wd = np.ascontiguousarray(np.asarray(wd, np.float64))
    H, I = wd.shape
    return O.expert_ffn(x, wg, wu, wd.reshape(I, H).T)


def _unnormalised_weights(p, idx, norm):
    return np.array([p[e] for e in idx], dtype=np.float64)


def _weight_ignored(cfg, T, slot, w):
    return O.slot_row_weight(cfg, T, slot, w)[0], 1.0


@pytest.mark.parametrize("repl", [
    dict(expert_ffn=_swap_gate_up), dict(expert_ffn=_no_sigmoid_scale), dict(expert_ffn=_transposed_down),
    dict(routing_weights=_unnormalised_weights), dict(slot_row_weight=_weight_ignored),
], ids=["swap_gate_up", "sigmoid_not_silu", "down_wrong", "weights_not_renormalised", "combine_ignores_weight"])
def test_planted_mistakes_are_caught(repl):
    assert _fails(PINS, _Mutant(**repl))
    assert not _fails(PINS, O)
