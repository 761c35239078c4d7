"""GPU parity: the CUDA library against the oracle, through the C ABI, on seeded workloads."""
import numpy as np
import pytest
import torch

from oracle import team_oracle as O
from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import workloads as W
from tests import _parity as P

pytestmark = pytest.mark.gpu

ALL_FLAGS = [0, B.TEAM_F_DCD, B.TEAM_F_LAC, B.TEAM_F_DCD | B.TEAM_F_LAC]


@pytest.fixture(scope="module")
def weights_cache():
    cache = {}

    def get(shape):
        key = (shape.hidden, shape.n_experts, shape.inter, shape.n_shared, shape.dtype, shape.seed)
        if key not in cache:
            cache[key] = W.make_weights(shape)
        return cache[key]
    return get


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_pack_w_down_is_the_stated_permutation(dtype):
    n, H, I = 3, 40, 48
    gen = torch.Generator().manual_seed(5)
    src = torch.randn((n, H, I), generator=gen).to(dtype)
    expected = src.view(n, H, I // 16, 16).permute(0, 2, 1, 3).contiguous()       # [n, I/16, H, 16]
    got = B.team_pack_w_down(src.cuda())
    torch.cuda.synchronize()
    assert got.shape == src.shape and got.dtype == dtype
    assert torch.equal(got.cpu().view(n, I // 16, H, 16), expected)


@pytest.mark.parametrize("flags", ALL_FLAGS)
def test_c1_tiny_fp32_all_steps(flags, weights_cache):
    stats = P.run_schedule(W.C1, weights_cache(W.C1), W.make_schedule(W.C1), flags)
    assert len(stats) == 8 and all(s["exact"] for s in stats)
    assert max(s["rel_err"] for s in stats) <= P.TOL_F32


@pytest.mark.parametrize("flags", ALL_FLAGS)
@pytest.mark.parametrize("shape", [W.MINI_BF16, W.MINI_SHARED, W.MINI_WRAP], ids=lambda s: s.name)
def test_mini_bf16_tensor_path(shape, flags, weights_cache):
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags)
    # router, selection, then gather + the two grouped GEMMs; the selection is two launches (rounds per group, then
    # dispatch) for several groups with more than 32 rows
    assert all(s["launches"] == (6 if shape.seqs > 1 and shape.rows > 32 else 5) for s in stats)


@pytest.mark.parametrize("shape", [W.MINI_BF16, W.MINI_SHARED], ids=lambda s: s.name)
def test_mini_bf16_fma_diagnostic_path(shape, weights_cache):
    P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), 3, force_simt=True)


@pytest.mark.parametrize("flags", [0, 1, 3])
def test_c2_sdar_shape(flags, weights_cache):
    stats = P.run_schedule(W.C2, weights_cache(W.C2), W.make_schedule(W.C2), flags)
    assert len(stats) == 4
    if flags == 3:
        assert [s["rows"] for s in stats] == [4, 4, 3, 2]


@pytest.mark.parametrize("flags", [0, 1, 3])
def test_few_rows_kernel_multi_pass_ranges_and_shared_expert(flags, weights_cache):
    shape = W.STREAM_MULTI
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags)
    assert len(stats) == 4
    if flags == 0:
        # enough activated experts that a CTA's range of column groups exceeds one pass (8 groups)
        assert max(s["n_active"] for s in stats) * (shape.inter // 16) > 8 * 148


@pytest.mark.parametrize("flags", [0, 3])
def test_few_rows_kernel_resident_mode_at_its_limits(flags, weights_cache):
    shape = W.STREAM_WIDE                        # 128 slots, 258 experts: every word of the activated bit set is used
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags)
    assert len(stats) == 3


@pytest.mark.parametrize("flags", [0, 3])
def test_few_rows_kernel_gather_mode_with_split_items(flags, weights_cache):
    shape = W.STREAM_GATHER                      # 24 rows: the shared expert alone has three items of 8 slots
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags)
    assert len(stats) == 4 and all(s["launches"] == 3 for s in stats)


@pytest.mark.parametrize("flags", [0, 3])
def test_few_rows_kernel_gather_mode_items_of_16_slots(flags, weights_cache):
    shape = W.STREAM_GATHER16                    # 80 rows in 2 groups: items of 16 slots, the shared expert has five
    stats = P.run_schedule(shape, weights_cache(shape), W.make_schedule(shape), flags,
                           knobs=[(B.TEAM_KNOB_EXPERT_KERNEL, 1)])      # (64 rows and more default to the tensor-memory kernels)
    # 40 rows per group are more than a CTA routes at once: the selection is one launch of a 2-CTA cluster
    assert len(stats) == 4 and all(s["launches"] == 3 for s in stats)


@pytest.mark.parametrize("flags", [0, 3])
def test_c3_llada_shape_with_shared_expert(flags, weights_cache):
    stats = P.run_schedule(W.C3, weights_cache(W.C3), W.make_schedule(W.C3), flags)
    assert len(stats) == 8


KERNELS = {"default": [], "streaming": [(B.TEAM_KNOB_EXPERT_KERNEL, 1)], "tensor_memory": [(B.TEAM_KNOB_EXPERT_KERNEL, 2)]}


@pytest.mark.parametrize("kernel", ["streaming", "tensor_memory"])
def test_paper_operating_point_block32_four_branches_one_group(weights_cache, kernel):
    shape = W.paper_point()                      # 128 rows, one group: cluster selection, one expert sees up to 108 slots
    steps = W.make_schedule(shape)[1:4]
    P.run_schedule(shape, weights_cache(shape), steps, 3, knobs=KERNELS[kernel])


@pytest.mark.parametrize("kernel", ["streaming", "tensor_memory"])
@pytest.mark.parametrize("seqs", [1, 4, 16, 64])
def test_c4_batch_sweep(seqs, weights_cache, kernel):
    shape = W.c4(seqs)
    steps = W.make_schedule(shape)
    # all four steps for the small batches, two for the large ones (the oracle takes seconds per step there)
    steps = steps if seqs <= 4 else steps[1:3]
    stats = P.run_schedule(shape, weights_cache(shape), steps, 3, knobs=KERNELS[kernel])
    assert all(s["launches"] >= (5 if kernel == "tensor_memory" else 3) for s in stats)
    if seqs <= 4:
        P.run_schedule(shape, weights_cache(shape), steps, 0, knobs=KERNELS[kernel])


@pytest.mark.parametrize("flags", [0, 3])
def test_c3_llada_shape_on_the_tensor_memory_kernels(flags, weights_cache):
    stats = P.run_schedule(W.C3, weights_cache(W.C3), W.make_schedule(W.C3)[:4], flags, knobs=KERNELS["tensor_memory"])
    assert all(s["launches"] == 5 for s in stats)


def test_tensor_memory_kernels_with_more_slots_than_a_chunk_holds(weights_cache):
    """An expert chosen by more than 128 token-slots is split into several chunks (its weights are then streamed
    once per chunk): 160 rows with a shared expert that every row uses."""
    import dataclasses
    shape = dataclasses.replace(W.STREAM_GATHER16, name="tile_split_chunks", block=40, seqs=4, seed=21)
    steps = W.make_schedule(shape)[:2]
    P.run_schedule(shape, weights_cache(shape), steps, 0, knobs=KERNELS["tensor_memory"])


def test_pack_w_tiles_is_the_stated_permutation():
    n, H, I = 2, 256, 128
    gen = torch.Generator().manual_seed(6)
    wg, wu = [torch.randn((n, I, H), generator=gen).to(torch.bfloat16) for _ in range(2)]
    wd = torch.randn((n, H, I), generator=gen).to(torch.bfloat16)
    gu, dt = B.team_pack_w_tiles(wg.cuda(), wu.cuda(), wd.cuda())
    torch.cuda.synchronize()
    gu = gu.cpu().view(torch.int16).numpy().reshape(n, I // 64, H // 64, 128, 8, 8)
    dt = dt.cpu().view(torch.int16).numpy().reshape(n, H // 128, I // 64, 128, 8, 8)
    g16, u16, d16 = (t.view(torch.int16).numpy() for t in (wg, wu, wd))
    for e in range(n):
        for u in range(I // 64):
            for kb in range(H // 64):
                for r in range(128):
                    blk, m, i = r // 32, (r // 16) % 2, r % 16
                    src = (u16 if m else g16)[e, u * 64 + blk * 16 + i, kb * 64:(kb + 1) * 64].reshape(8, 8)
                    for p in range(8):
                        np.testing.assert_array_equal(gu[e, u, kb, r, p ^ (r & 7)], src[p])
        for ht in range(H // 128):
            for kb in range(I // 64):
                for r in range(128):
                    src = d16[e, ht * 128 + r, kb * 64:(kb + 1) * 64].reshape(8, 8)
                    for p in range(8):
                        np.testing.assert_array_equal(dt[e, ht, kb, r, p ^ (r & 7)], src[p])


def _run_stack(shape, n_layers, flags, weights_cache, tables=True):
    """MoE-only stack (config 5's structure): x <- x + layer(x) on computed rows, layer after layer, step after step.

    Every layer is checked teacher-forced (the oracle gets the activations the GPU stack actually fed into that
    layer, which are exact in the storage type), so a near-tie early in the stack cannot cascade; the stack's final
    activations are compared with the oracle's own stack as well.
    """
    import dataclasses
    layers_w = [W.make_weights(dataclasses.replace(shape, seed=shape.seed + 100 * l)) for l in range(n_layers)]
    steps = W.make_schedule(shape)
    ocfg = P.oracle_config(shape, flags)
    layers = [P.Layer(shape, w, flags) for w in layers_w]
    dc = P.dtype_code(shape)
    T = steps[0]["x"].shape[0]
    round_fn = (lambda a: W.round_to_bf16(np.asarray(a, dtype=np.float32)).astype(np.float64)) if shape.dtype == "bf16" \
        else (lambda a: np.asarray(a, dtype=np.float32).astype(np.float64))
    try:
        for si, step in enumerate(steps):
            x_dev = B.to_device(step["x"], dc)
            st = B.state_to_device(step)
            y_dev = torch.zeros((T, shape.hidden), dtype=torch.float32, device="cuda")
            all_exact = True
            for li, layer in enumerate(layers):
                x_in = x_dev.float().cpu().numpy()
                out = B.alloc_routing(layer.cfg, T)
                if not tables:
                    out = {n: out[n] for n in P.CHOICE_TABLES}
                y_before = y_dev.cpu().numpy()
                B.team_moe_forward(layer.ctx, x_dev, st, out, y_dev)
                B.team_residual_add(layer.ctx, x_dev, y_dev, T)
                code, detail = B.team_read_status(layer.ctx)
                assert code == B.TEAM_OK, (code, detail)
                got = B.routing_to_host(out)
                if not tables:
                    got["n_rows_active"] = int((got["tok_class"] != O.CLS_SKIP).sum())
                y_ref, ref = O.moe_forward(ocfg, layers_w[li], x_in, step["tok_state"], step["conf"], step["pos"],
                                           step["group"], step["branch"], y_prev=y_before)
                what = f"{shape.name} stack step={si} layer={li}"
                exact, pin = P.compare_routing(ocfg, ref, got, step["group"], what, return_pin=True)
                all_exact = all_exact and exact
                P.compare_y_rows(shape, ocfg, layers_w[li], x_in, y_ref, ref, got, y_dev.cpu().numpy(), pin, y_before, what,
                                 max_unpinned=max(1, T // 32))      # inputs of deeper layers come from the stack itself
                # the residual add: fp32 add, stored in the activation type
                comp = ref["tok_class"] != O.CLS_SKIP
                want = x_in.astype(np.float64).copy()
                want[comp] = round_fn(x_in[comp].astype(np.float32) + y_dev.cpu().numpy()[comp])
                np.testing.assert_array_equal(x_dev.float().cpu().numpy().astype(np.float64), want, err_msg=what)
            if all_exact:
                x_ref, _ = O.stack_forward(ocfg, layers_w, step["x"], step["tok_state"], step["conf"], step["pos"],
                                           step["group"], step["branch"], round_fn=round_fn)
                x_got = x_dev.float().cpu().numpy()
                tol = (P.TOL_BF16 if shape.dtype == "bf16" else P.TOL_F32) * np.abs(x_ref).max()
                assert np.abs(x_got - x_ref).max() <= tol * n_layers, f"{shape.name} stack step={si} end to end"
    finally:
        for layer in layers:
            layer.close()


@pytest.mark.parametrize("flags", [0, 3])
def test_c5_stack_small_shape(flags, weights_cache):
    _run_stack(W.MINI_WRAP, 8, flags, weights_cache)


@pytest.mark.parametrize("tables", [True, False], ids=["three_kernels", "one_kernel_step"])
def test_c5_stack_sdar_shape_two_layers(weights_cache, tables):
    _run_stack(W.C2, 2, 3, weights_cache, tables=tables)


@pytest.mark.parametrize("side_stream", [False, True], ids=["default_stream", "own_stream_graph_replay"])
def test_host_buffer_entry_point_matches_device_entry_point(side_stream, weights_cache):
    """team_moe_forward_host on a whole schedule, twice over (on a stream of its own the library replays the
    recorded step from the second call on): same y as team_moe_forward, skipped rows keeping the previous step's."""
    shape, flags = W.C2, 3
    steps = W.make_schedule(shape) * 2
    if side_stream:
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            _host_entry_schedule(shape, flags, steps, weights_cache)
        torch.cuda.current_stream().wait_stream(stream)
    else:
        _host_entry_schedule(shape, flags, steps, weights_cache)


def _host_entry_schedule(shape, flags, steps, weights_cache):
    layer_a, layer_b = P.Layer(shape, weights_cache(shape), flags), P.Layer(shape, weights_cache(shape), flags)
    try:
        T, H = shape.rows, shape.hidden
        y_dev = torch.zeros((T, H), dtype=torch.float32, device="cuda")
        y_host = torch.full((T, H), 7.0, dtype=torch.float32)
        for step in steps:
            x_host = torch.as_tensor(step["x"]).to(torch.bfloat16)
            st_host = {"tok_state": torch.as_tensor(step["tok_state"].astype(np.uint8)),
                       "conf": torch.as_tensor(step["conf"].astype(np.float32)),
                       "pos": torch.as_tensor(step["pos"].astype(np.int32)),
                       "group": torch.as_tensor(step["group"].astype(np.int32)),
                       "branch": torch.as_tensor(step["branch"].astype(np.int32))}
            B.team_moe_forward(layer_a.ctx, x_host.cuda(), B.state_to_device(step), None, y_dev)
            B.team_moe_forward_host(layer_b.ctx, x_host, st_host, None, y_host)
            ref = y_dev.cpu()
            # fp32 reductions arrive in a different order from launch to launch: equal to rounding of the sums
            assert torch.allclose(y_host, ref, rtol=0, atol=1e-5 * float(ref.abs().max()))
        assert B.team_read_status(layer_b.ctx)[0] == 0
    finally:
        layer_a.close()
        layer_b.close()


@pytest.mark.parametrize("shape", [W.C2, W.STREAM_MULTI, W.STREAM_WIDE], ids=lambda s: s.name)
def test_forward_without_exports_skips_the_dispatch_tables_and_gives_the_same_y(shape, weights_cache):
    """With at most 8 rows and no table asked for, the selection stops after the routing rounds and the expert
    kernel works from the rows' choices; y must not depend on that."""
    steps = W.make_schedule(shape)
    for flags in (0, 3):
        layer_a, layer_b = P.Layer(shape, weights_cache(shape), flags), P.Layer(shape, weights_cache(shape), flags)
        try:
            T, H = shape.rows, shape.hidden
            y_a = torch.zeros((T, H), dtype=torch.float32, device="cuda")
            y_b = torch.zeros((T, H), dtype=torch.float32, device="cuda")
            for step in steps:
                x = B.to_device(step["x"], B.TEAM_DTYPE_BF16)
                st = B.state_to_device(step)
                out = B.alloc_routing(layer_a.cfg, T)
                B.team_moe_forward(layer_a.ctx, x, st, out, y_a)          # all tables exported
                B.team_moe_forward(layer_b.ctx, x, st, None, y_b)         # none
                torch.cuda.synchronize()
                assert int(out["n_active"].item()) > 0
                assert torch.allclose(y_b, y_a, rtol=0, atol=1e-5 * float(y_a.abs().max()))
            assert B.team_read_status(layer_b.ctx)[0] == 0
        finally:
            layer_a.close()
            layer_b.close()
