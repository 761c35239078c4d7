"""ctypes binding of libteam_b200.so (the C ABI declared in include/team.h).

Argument marshalling only: torch supplies device memory and the current CUDA
stream; every step of the layer runs in the library's kernels.  There is no
fallback: if the library has not been built, or no CUDA device is usable,
calls raise.
"""
import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libteam_b200.so")

TEAM_OK, TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA, TEAM_ERR_TIMEOUT, TEAM_ERR_STATE = 0, -1, -2, -3, -4, -5
TEAM_ERR_CAPACITY = -6
TEAM_STATIC_ROUTE_MAX_ROWS = 256
TEAM_TOK_MASKED, TEAM_TOK_NEW, TEAM_TOK_CACHED = 0, 1, 2
TEAM_CLS_SKIP, TEAM_CLS_FIRST, TEAM_CLS_COLD = 0, 1, 2
TEAM_F_DCD, TEAM_F_LAC = 1, 2
TEAM_DTYPE_F32, TEAM_DTYPE_BF16 = 0, 1

EXPORTS = ["team_create", "team_destroy", "team_set_weights", "team_set_policy", "team_route",
           "team_route_static", "team_pack_w_down", "team_pack_w_tiles", "team_seh_step", "team_block_attention", "team_select_experts", "team_moe_forward", "team_moe_forward_host", "team_residual_add", "team_read_status",
           "team_last_launch_count", "team_expert_kernel_name", "team_expert_timing", "team_debug_force_simt", "team_debug_knob", "team_strerror",
           "team_last_cuda_error", "team_version"]


class team_config(ctypes.Structure):
    _fields_ = [("hidden", ctypes.c_int32), ("n_experts", ctypes.c_int32), ("top_k", ctypes.c_int32),
                ("inter", ctypes.c_int32), ("n_shared", ctypes.c_int32), ("max_rows", ctypes.c_int32),
                ("max_groups", ctypes.c_int32), ("dtype", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("tau_hot", ctypes.c_float), ("L_hot", ctypes.c_int32), ("hot_dist_inclusive", ctypes.c_int32),
                ("prefix_decoded", ctypes.c_int32), ("norm_topk", ctypes.c_int32), ("refresh_every", ctypes.c_int32),
                ("ep_rank", ctypes.c_int32), ("ep_world", ctypes.c_int32)]


class team_weights(ctypes.Structure):
    _fields_ = [("w_router", ctypes.c_void_p), ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p),
                ("w_down", ctypes.c_void_p), ("w_gu_tiles", ctypes.c_void_p), ("w_down_tiles", ctypes.c_void_p)]


class team_step_state(ctypes.Structure):
    _fields_ = [("n_rows", ctypes.c_int32), ("tok_state", ctypes.c_void_p), ("conf", ctypes.c_void_p),
                ("pos", ctypes.c_void_p), ("group", ctypes.c_void_p), ("branch", ctypes.c_void_p),
                ("step_index", ctypes.c_int32)]


class team_seh_config(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("block", ctypes.c_int32), ("n_branches", ctypes.c_int32),
                ("tau", ctypes.c_float)]


class team_seh_state(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("token", "state", "spec_pos", "spec_tok", "counters")]


class team_seh_rows(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("tok_state", "conf", "pos", "group", "branch")]


class team_attn_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_heads", "n_kv_heads", "head_dim", "block", "n_seqs", "n_branches",
                                               "max_prefix", "flags")]


class team_routing(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("probs", "topk_idx", "topk_w", "margin", "tok_class", "group_mask", "expert_count",
                 "expert_offset", "perm", "active", "n_active", "n_rows_active")]


_lib_handle = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib_handle
    if _lib_handle is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_08404_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32 = ctypes.c_void_p, ctypes.c_int32
        L.team_create.argtypes = [ctypes.POINTER(team_config), ctypes.POINTER(vp)]
        L.team_destroy.argtypes = [vp]
        L.team_set_weights.argtypes = [vp, ctypes.POINTER(team_weights)]
        L.team_set_policy.argtypes = [vp, ctypes.POINTER(team_config)]
        L.team_route.argtypes = [vp, vp, ctypes.POINTER(team_step_state), ctypes.POINTER(team_routing), vp]
        L.team_pack_w_down.argtypes = [vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp]
        L.team_pack_w_tiles.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp]
        L.team_seh_step.argtypes = [ctypes.POINTER(team_seh_config), ctypes.POINTER(team_seh_state), vp, vp,
                                    ctypes.POINTER(team_seh_rows), vp, vp]
        L.team_block_attention.argtypes = [ctypes.POINTER(team_attn_config), ctypes.POINTER(team_step_state)] + [vp] * 11
        L.team_route_static.argtypes = [ctypes.POINTER(team_config), vp, vp, ctypes.POINTER(team_step_state),
                                        ctypes.POINTER(team_routing), vp]
        L.team_select_experts.argtypes = [vp, ctypes.POINTER(team_step_state), ctypes.POINTER(team_routing), vp]
        L.team_moe_forward.argtypes = [vp, vp, ctypes.POINTER(team_step_state), ctypes.POINTER(team_routing), vp, vp]
        L.team_moe_forward_host.argtypes = [vp, vp, ctypes.POINTER(team_step_state), ctypes.POINTER(team_routing), vp, vp]
        L.team_residual_add.argtypes = [vp, vp, vp, i32, vp]
        L.team_read_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.team_last_launch_count.argtypes = [vp]
        L.team_expert_timing.argtypes = [vp, i32, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
        L.team_debug_force_simt.argtypes = [vp, i32]
        L.team_debug_knob.argtypes = [vp, i32, ctypes.c_longlong]
        L.team_strerror.argtypes = [i32]
        L.team_strerror.restype = ctypes.c_char_p
        L.team_expert_kernel_name.argtypes = [vp]
        L.team_expert_kernel_name.restype = ctypes.c_char_p
        L.team_last_cuda_error.argtypes = [vp]
        L.team_last_cuda_error.restype = ctypes.c_char_p
        for name in EXPORTS:
            if getattr(L, name).restype is not ctypes.c_char_p:
                getattr(L, name).restype = ctypes.c_int
        _lib_handle = L
    return _lib_handle


class TeamError(RuntimeError):
    pass


def _check(rc, ctx=None):
    if rc != TEAM_OK:
        msg = lib().team_strerror(rc).decode()
        if ctx is not None and rc == TEAM_ERR_CUDA:
            msg += ": " + lib().team_last_cuda_error(ctx).decode()
        raise TeamError(f"team error {rc}: {msg}")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise TeamError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(hidden, n_experts, top_k, inter, n_shared=0, max_rows=64, max_groups=1, dtype=TEAM_DTYPE_BF16,
                flags=0, tau_hot=0.7, L_hot=3, hot_dist_inclusive=1, prefix_decoded=1, norm_topk=1, refresh_every=0, ep_rank=0, ep_world=1):
    return team_config(hidden, n_experts, top_k, inter, n_shared, max_rows, max_groups, dtype, flags, tau_hot,
                       L_hot, hot_dist_inclusive, prefix_decoded, norm_topk, refresh_every, ep_rank, ep_world)


# ---- the C entry points, same names, torch tensors for device memory ---------------------------------
def team_create(cfg):
    if not torch.cuda.is_available():
        raise TeamError("no CUDA device: the TEAM library has no CPU path")
    ctx = ctypes.c_void_p()
    _check(lib().team_create(ctypes.byref(cfg), ctypes.byref(ctx)))
    return ctx


def team_destroy(ctx):
    _check(lib().team_destroy(ctx))


def team_set_weights(ctx, w_router, w_gate=None, w_up=None, w_down=None, w_gu_tiles=None, w_down_tiles=None):
    """w_gate / w_up / w_down: the row-major / slab layout; w_gu_tiles / w_down_tiles: the tile-major layout."""
    w = team_weights(_ptr(w_router), _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(w_gu_tiles), _ptr(w_down_tiles))
    _check(lib().team_set_weights(ctx, ctypes.byref(w)), ctx)


def team_pack_w_tiles(w_gate, w_up, w_down):
    """Row-major bf16 device tensors [n, I, H], [n, I, H], [n, H, I] -> (gu_tiles, down_tiles) in the tile-major layout."""
    n, I, H = w_gate.shape
    gu = torch.empty((2 * n * I * H,), dtype=torch.bfloat16, device=w_gate.device)
    dt = torch.empty((n * I * H,), dtype=torch.bfloat16, device=w_gate.device)
    _check(lib().team_pack_w_tiles(_ptr(w_gate.contiguous()), _ptr(w_up.contiguous()), _ptr(w_down.contiguous()), _ptr(gu),
                                   _ptr(dt), n, H, I, _stream()))
    return gu, dt


def team_pack_w_down(w_down):
    """Row-major [n_experts_total, H, I] device tensor -> new tensor in the slab layout team_set_weights expects."""
    n, H, I = w_down.shape
    dtype = TEAM_DTYPE_BF16 if w_down.dtype == torch.bfloat16 else TEAM_DTYPE_F32
    src = w_down.contiguous()
    dst = torch.empty_like(src)
    _check(lib().team_pack_w_down(_ptr(src), _ptr(dst), n, H, I, dtype, _stream()))
    return dst


def team_set_policy(ctx, cfg):
    _check(lib().team_set_policy(ctx, ctypes.byref(cfg)), ctx)


def _state(st):
    return team_step_state(int(st["tok_state"].shape[0]), _ptr(st["tok_state"]), _ptr(st["conf"]), _ptr(st["pos"]),
                           _ptr(st["group"]), _ptr(st["branch"]), int(st.get("step_index", 0)))


def _routing(out):
    if out is None:
        return None
    return team_routing(*[_ptr(out.get(n)) for n, _ in team_routing._fields_])


def team_route(ctx, x, st, out):
    r = _routing(out)
    _check(lib().team_route(ctx, _ptr(x), ctypes.byref(_state(st)), ctypes.byref(r), _stream()), ctx)


def team_route_static(cfg, x, w_router, st, out):
    """Router step with no context and no allocation (fixed scratch inside the library); returns the status code
    instead of raising so that callers can test the capacity limit."""
    r = _routing(out)
    return lib().team_route_static(ctypes.byref(cfg), _ptr(x), _ptr(w_router), ctypes.byref(_state(st)), ctypes.byref(r),
                                   _stream())


def seh_alloc(n_seqs, block, n_branches=4, device="cuda"):
    """Device buffers of the decode-loop glue: (state dict, rows dict) as team_seh_step takes them."""
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
    T = n_seqs * n_branches * block
    state = dict(token=z((n_seqs, block), torch.int32), state=z((n_seqs, block), torch.uint8),
                 spec_pos=z((n_seqs, 2), torch.int32), spec_tok=z((n_seqs, 2), torch.int32), counters=z((n_seqs, 2), torch.int32))
    rows = dict(tok_state=z((T,), torch.uint8), conf=z((T,), torch.float32), pos=z((T,), torch.int32),
                group=z((T,), torch.int32), branch=z((T,), torch.int32))
    return state, rows


def team_seh_step(n_seqs, block, n_branches, tau, state, pred, conf, rows, adopted=None):
    """pred / conf: device tensors [S, n_branches, L] (both None: begin a block)."""
    cfg = team_seh_config(n_seqs, block, n_branches, tau)
    st = team_seh_state(*[_ptr(state[n]) for n, _ in team_seh_state._fields_])
    rw = team_seh_rows(*[_ptr(rows[n]) for n, _ in team_seh_rows._fields_])
    _check(lib().team_seh_step(ctypes.byref(cfg), ctypes.byref(st), _ptr(pred), _ptr(conf), ctypes.byref(rw), _ptr(adopted),
                               _stream()))


def team_block_attention(cfg, st, q, k_new, v_new, k_prefix, v_prefix, prefix_len, k_block, v_block, out, status=None):
    """cfg: team_attn_config; st: dict of device tensors (tok_state, pos, group, branch; conf is not read)."""
    T = int(st["tok_state"].shape[0])
    s = team_step_state(T, _ptr(st["tok_state"]), _ptr(st.get("conf")), _ptr(st["pos"]), _ptr(st["group"]), _ptr(st["branch"]), 0)
    return lib().team_block_attention(ctypes.byref(cfg), ctypes.byref(s), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_prefix),
                                      _ptr(v_prefix), _ptr(prefix_len), _ptr(k_block), _ptr(v_block), _ptr(out), _ptr(status),
                                      _stream())


def team_select_experts(ctx, st, out):
    r = _routing(out)
    _check(lib().team_select_experts(ctx, ctypes.byref(_state(st)), ctypes.byref(r) if r is not None else None, _stream()), ctx)


def team_moe_forward(ctx, x, st, out, y):
    r = _routing(out)
    _check(lib().team_moe_forward(ctx, _ptr(x), ctypes.byref(_state(st)), ctypes.byref(r) if r is not None else None, _ptr(y),
                                  _stream()), ctx)


def _hptr(t):
    if t.is_cuda or not t.is_contiguous():
        raise TeamError("expected a contiguous CPU tensor")
    return ctypes.c_void_p(t.data_ptr())


def team_moe_forward_host(ctx, x_host, st_host, out, y_host):
    """x_host, the step state and y_host are CPU tensors; `out` (optional) holds device tensors. Blocks until y_host is filled."""
    st = team_step_state(int(st_host["tok_state"].shape[0]), _hptr(st_host["tok_state"]), _hptr(st_host["conf"]),
                         _hptr(st_host["pos"]), _hptr(st_host["group"]), _hptr(st_host["branch"]),
                         int(st_host.get("step_index", 0)))
    r = _routing(out)
    _check(lib().team_moe_forward_host(ctx, _hptr(x_host), ctypes.byref(st), ctypes.byref(r) if r is not None else None,
                                       _hptr(y_host), _stream()), ctx)


def team_residual_add(ctx, x, y, n_rows):
    _check(lib().team_residual_add(ctx, _ptr(x), _ptr(y), int(n_rows), _stream()), ctx)


def team_read_status(ctx):
    detail = ctypes.c_int32(0)
    code = lib().team_read_status(ctx, _stream(), ctypes.byref(detail))
    return code, detail.value


def team_last_launch_count(ctx):
    return lib().team_last_launch_count(ctx)


def team_expert_kernel_name(ctx):
    return lib().team_expert_kernel_name(ctx).decode()


def team_expert_timing(ctx, enable):
    ms, n = ctypes.c_float(0), ctypes.c_int32(0)
    _check(lib().team_expert_timing(ctx, int(enable), _stream(), ctypes.byref(ms), ctypes.byref(n)), ctx)
    return ms.value, n.value


TEAM_KNOB_NO_FUSE, TEAM_KNOB_EXTRA_ARRIVALS, TEAM_KNOB_WAIT_LIMIT_US, TEAM_KNOB_EXPERT_KERNEL = 1, 2, 3, 4
TEAM_KNOB_ORDERED_COMBINE = 5


def team_debug_knob(ctx, knob, value):
    _check(lib().team_debug_knob(ctx, int(knob), int(value)), ctx)


def team_debug_force_simt(ctx, on):
    _check(lib().team_debug_force_simt(ctx, int(on)), ctx)


# ---- convenience: device buffers for the routing tables and the step state ----------------------------
def alloc_routing(cfg, n_rows, device="cuda"):
    T, E, k, ns = n_rows, cfg.n_experts, cfg.top_k, cfg.n_shared
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
    return dict(probs=z((T, E), torch.float32), topk_idx=z((T, k), torch.int32), topk_w=z((T, k), torch.float32),
                margin=z((T,), torch.float32), tok_class=z((T,), torch.uint8),
                group_mask=z((cfg.max_groups, (E + 63) // 64), torch.int64),
                expert_count=z((E + ns,), torch.int32), expert_offset=z((E + ns + 1,), torch.int32),
                perm=z((T * (k + ns),), torch.int32), active=z((E + ns,), torch.int32),
                n_active=z((1,), torch.int32), n_rows_active=z((1,), torch.int32))


def routing_to_host(out):
    r = {n: v.cpu().numpy() for n, v in out.items()}
    if "group_mask" in r:
        r["group_mask"] = r["group_mask"].view(np.uint64)
    if "n_active" in r:
        r["n_active"] = int(r["n_active"][0])
        r["n_rows_active"] = int(r["n_rows_active"][0])
        r["active"] = r["active"][:r["n_active"]]
    return r


def state_to_device(step, device="cuda"):
    return dict(tok_state=torch.as_tensor(np.asarray(step["tok_state"], dtype=np.uint8)).to(device),
                conf=torch.as_tensor(np.asarray(step["conf"], dtype=np.float32)).to(device),
                pos=torch.as_tensor(np.asarray(step["pos"], dtype=np.int32)).to(device),
                group=torch.as_tensor(np.asarray(step["group"], dtype=np.int32)).to(device),
                branch=torch.as_tensor(np.asarray(step["branch"], dtype=np.int32)).to(device))


def to_device(a, dtype_code, device="cuda"):
    """fp32 host array (values exact in the storage type) -> device tensor in the storage type."""
    t = torch.as_tensor(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return t.to(torch.bfloat16).contiguous() if dtype_code == TEAM_DTYPE_BF16 else t.contiguous()
