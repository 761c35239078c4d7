"""team_route_static: the router step for callers that are not allowed to allocate device memory.

Some users of this library run where cudaMalloc is forbidden: a serving loop whose device memory was
planned and frozen at start-up, a plug-in invoked from inside someone else's stream capture or
callback, or a latency-critical path that cannot afford the allocator's implicit synchronisation.
They cannot create a context (team_create allocates the logits workspace), so the library offers one
entry point that keeps the logits in a fixed 256 KiB array inside the library image instead.

The test calls it through the C ABI twice in a row (the array is shared by all calls and keeps the
previous call's contents) and compares every output with team_route on a regular context (both run
the same kernels, so integer outputs must be identical and floating-point outputs equal to rounding)
and with the CPU oracle's router and top-k.  It also watches the device's free memory and torch's
allocator across a series of calls: neither may move.
The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _route_both(shape, step, flags):
    """Outputs of team_route (context) and of two successive team_route_static calls on one step."""
    dc = B.TEAM_DTYPE_BF16 if shape.dtype == "bf16" else B.TEAM_DTYPE_F32
    T = step["x"].shape[0]
    cfg = B.make_config(shape.hidden, shape.n_experts, shape.top_k, shape.inter, shape.n_shared, max_rows=T,
                        max_groups=shape.seqs, dtype=dc, flags=flags, tau_hot=shape.tau_hot, L_hot=shape.L_hot)
    weights = W.make_weights(shape)
    w_router = torch.as_tensor(weights["w_router"]).cuda().contiguous()
    x = B.to_device(step["x"], dc)
    st = B.state_to_device(step)
    names = ("probs", "topk_idx", "topk_w", "margin")

    ctx = B.team_create(cfg)
    try:
        B.team_set_weights(ctx, w_router, B.to_device(weights["w_gate"], dc), B.to_device(weights["w_up"], dc),
                           B.team_pack_w_down(B.to_device(weights["w_down"], dc)))
        ref = B.alloc_routing(cfg, T)
        B.team_route(ctx, x, st, ref)
        torch.cuda.synchronize()
        ref = {n: ref[n].cpu().numpy() for n in names}
    finally:
        B.team_destroy(ctx)

    got = []
    for _ in range(2):
        out = B.alloc_routing(cfg, T)
        for n in names:                       # poison: the call must write every element it owns
            out[n].fill_(-7)
        rc = B.team_route_static(cfg, x, w_router, st, out)
        assert rc == B.TEAM_OK, B.lib().team_strerror(rc)
        torch.cuda.synchronize()
        got.append({n: out[n].cpu().numpy() for n in names})
    return ref, got


def _oracle_route(shape, step, flags):
    """Softmax table, plain top-k, weights and margin of every computed row from the oracle's pieces."""
    weights = W.make_weights(shape)
    logits32, probs = O.router(step["x"], weights["w_router"])
    T, k = logits32.shape[0], shape.top_k
    computed = np.zeros(T, dtype=bool)
    computed[O.active_rows(step["tok_state"], flags)] = True
    idx, w, margin = np.full((T, k), -1), np.zeros((T, k)), np.full(T, np.inf)
    clear = np.zeros(T, dtype=bool)
    for t in np.flatnonzero(computed):
        take, margin[t] = O.topk_row(logits32[t], k)
        idx[t], w[t] = take, O.routing_weights(probs[t], take, 1)
        order = np.sort(logits32[t].astype(np.float64))[::-1][:k + 1]
        clear[t] = np.min(-np.diff(order)) > 1e-5            # every ordering decision clearer than 1e-5
    return dict(probs=probs, topk_idx=idx, topk_w=w, margin=margin), computed, clear


@pytest.mark.parametrize("shape,flags", [(W.C2, 3), (W.C1, 1), (W.MINI_SHARED, 3), (W.c4(4), 0)],
                         ids=["c2_bf16", "c1_f32", "mini_shared", "c4_b4_64rows"])
def test_static_route_matches_context_route_twice_in_a_row(shape, flags):
    step = W.make_schedule(shape)[2]          # a step with cached, new and masked rows
    ref, got = _route_both(shape, step, flags)
    for g in got:
        np.testing.assert_array_equal(g["topk_idx"], ref["topk_idx"])
        np.testing.assert_allclose(g["topk_w"], ref["topk_w"], rtol=1e-6, atol=1e-7)
        np.testing.assert_allclose(g["probs"], ref["probs"], rtol=1e-6, atol=1e-9)
        np.testing.assert_array_equal(np.isinf(g["margin"]), np.isinf(ref["margin"]))
        fin = np.isfinite(ref["margin"])
        np.testing.assert_allclose(g["margin"][fin], ref["margin"][fin], rtol=1e-6, atol=1e-7)
    # ... and against the oracle, at the tolerances of the parity suite
    orc, computed, clear = _oracle_route(shape, step, flags)
    assert clear[computed].mean() >= 0.99
    for g in got:
        np.testing.assert_allclose(g["probs"][computed], orc["probs"][computed], rtol=0, atol=1e-6)
        assert not g["probs"][~computed].any() and (g["topk_idx"][~computed] == -1).all()
        for t in np.flatnonzero(computed & clear):
            np.testing.assert_array_equal(g["topk_idx"][t], orc["topk_idx"][t])
            np.testing.assert_allclose(g["topk_w"][t], orc["topk_w"][t], rtol=1e-5, atol=2e-6)
            assert abs(g["margin"][t] - orc["margin"][t]) < 1e-5 or np.isinf(orc["margin"][t])


def test_static_route_allocates_no_device_memory():
    """After one call has done the per-device set-up, further calls leave the device's free memory and torch's
    allocator exactly where they were."""
    shape = W.C2
    step = W.make_schedule(shape)[2]
    T = step["x"].shape[0]
    cfg = B.make_config(shape.hidden, shape.n_experts, shape.top_k, shape.inter, max_rows=T, flags=3)
    w_router = torch.as_tensor(W.make_weights(shape)["w_router"]).cuda().contiguous()
    x = B.to_device(step["x"], B.TEAM_DTYPE_BF16)
    st = B.state_to_device(step)
    out = B.alloc_routing(cfg, T)
    assert B.team_route_static(cfg, x, w_router, st, out) == B.TEAM_OK      # set-up happens here
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(20):
        assert B.team_route_static(cfg, x, w_router, st, out) == B.TEAM_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)


def test_static_route_rejects_a_hidden_size_its_kernels_cannot_stage():
    """The router kernels stage 8 rows of fp32 activations in shared memory; a hidden size beyond what one SM can
    hold is a shape error, reported before anything is launched."""
    cfg = B.make_config(16384, 64, 4, 768, max_rows=4)
    T = 4
    x = torch.zeros((T, 16384), dtype=torch.bfloat16, device="cuda")
    w_router = torch.zeros((64, 16384), dtype=torch.float32, device="cuda")
    st = dict(tok_state=torch.zeros(T, dtype=torch.uint8, device="cuda"), conf=torch.zeros(T, device="cuda"),
              pos=torch.zeros(T, dtype=torch.int32, device="cuda"), group=torch.zeros(T, dtype=torch.int32, device="cuda"),
              branch=torch.zeros(T, dtype=torch.int32, device="cuda"))
    assert B.team_route_static(cfg, x, w_router, st, B.alloc_routing(cfg, T)) == B.TEAM_ERR_SHAPE


def test_static_route_rejects_more_rows_than_its_scratch_holds():
    shape = W.C2
    T = B.TEAM_STATIC_ROUTE_MAX_ROWS + 1
    cfg = B.make_config(shape.hidden, shape.n_experts, shape.top_k, shape.inter, max_rows=2048)
    x = torch.zeros((T, shape.hidden), dtype=torch.bfloat16, device="cuda")
    w_router = torch.zeros((shape.n_experts, shape.hidden), dtype=torch.float32, device="cuda")
    st = dict(tok_state=torch.zeros(T, dtype=torch.uint8, device="cuda"), conf=torch.zeros(T, device="cuda"),
              pos=torch.zeros(T, dtype=torch.int32, device="cuda"), group=torch.zeros(T, dtype=torch.int32, device="cuda"),
              branch=torch.zeros(T, dtype=torch.int32, device="cuda"))
    out = B.alloc_routing(cfg, T)
    rc = B.team_route_static(cfg, x, w_router, st, out)
    assert rc == B.TEAM_ERR_CAPACITY
    assert b"scratch" in B.lib().team_strerror(rc)
    # exactly at the limit it runs
    T = B.TEAM_STATIC_ROUTE_MAX_ROWS
    st = {n: v[:T].contiguous() for n, v in st.items()}
    out = B.alloc_routing(cfg, T)
    assert B.team_route_static(cfg, x[:T].contiguous(), w_router, st, out) == B.TEAM_OK
    torch.cuda.synchronize()
    assert int(out["topk_idx"].min()) >= 0
