"""CPU oracle for the TEAM MoE-layer step.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain statement of what one MoE layer computes inside
one denoising step of a block-diffusion MoE language model when TEAM's expert
activation rule is applied.  It exists so that the CUDA library can be checked
against something that can be compared with the paper by eye.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import it; the
CUDA path shares no code with it.

Everything is numpy on the host.  Floating point is fp64 on exactly-widened
inputs, with one deliberate exception: the router logits are rounded to fp32
before any expert is chosen, because the method takes its top-k decisions on
an fp32 router and both sides must decide in the same precision.  Top-k is
taken on the logits (softmax is monotone, so the chosen set is the same as on
the probabilities and does not depend on how exp() rounds).

Steps, in the order of the paper:

  o1  rows computed this step         Sec. 4.1 (delayed caching, DCD)
  o2  router logits and softmax       Algorithm 1, "Router"
  o3  hot / cold classification       Eq. 4 and the text under it; Sec. 5.1
  o4  first-round rows                Algorithm 1, steps 1-2
  o5  first-round top-k               Algorithm 1, step 2
  o6  necessary expert set E_A        Algorithm 1, step 2; Sec. 4.3
  o7  second-round (restricted) top-k Algorithm 1, step 3
  o8  dispatch (counts, offsets, permutation, active list)
  o9  SwiGLU expert FFNs and the weighted combine
  o10 cached rows keep their previous output        Sec. 4.1

Readings taken where the paper is silent or garbled (each is a Config field or
stated where it is applied):

  * Eq. 4 prints "for all j"; the prose says a hot token is close to decoded
    tokens, so the distance test is "there exists a decoded position j".
  * Eq. 4 prints "<" while Sec. 5.1 says "no more than L_h positions away":
    hot_dist_inclusive=1 takes "<=" (default), 0 takes "<".
  * prefix_decoded=1 counts the last token of the previous block (position -1)
    as decoded, so the first step of a block has a hot token.
  * If a group has no first-round row at all, every masked row of that group
    is treated as hot (Algorithm 1 would otherwise produce an empty E_A).
  * E_A is the union of the per-token top-k sets of the first-round rows
    (Sec. 4.3), per caller-supplied group; decoded positions in Eq. 4 are
    scoped per (group, branch).
  * Router = softmax over all experts, weights renormalised over the k chosen
    (norm_topk=1).  Under renormalisation, masking to E_A before or after the
    softmax gives the same weights.
  * With DCD off, every decoded row (new or old) is computed and is a
    first-round row.
  * Shared experts (if any) are applied to every computed row with weight 1.
  * Periodic refresh (Sec. 4.1, second paragraph; Table 3, Refresh-4 / Refresh-8): with refresh_every = N > 0
    every N-th denoising step of a block (step_index 0, N, 2N, ...) recomputes all tokens -- on such a step a
    cached token is treated like a newly accepted one.  N = 0 is the paper's own choice, refresh-free.

Parity pins live in tests/test_oracle_*.py; every function below is pinned by
at least one of them.
"""

from dataclasses import dataclass

import numpy as np

TOK_MASKED, TOK_NEW, TOK_CACHED = 0, 1, 2
F_DCD, F_LAC = 1, 2
CLS_SKIP, CLS_FIRST, CLS_COLD = 0, 1, 2


@dataclass
class Config:
    hidden: int
    n_experts: int
    top_k: int
    inter: int
    n_shared: int = 0
    flags: int = 0
    tau_hot: float = 0.7
    L_hot: int = 3
    hot_dist_inclusive: int = 1
    prefix_decoded: int = 1
    norm_topk: int = 1
    max_groups: int = 1
    refresh_every: int = 0


# ----------------------------------------------------------------------------
# o1 -- Sec. 4.1: only masked tokens and tokens accepted in the previous step
# are computed; tokens decoded earlier are served from cache.
# ----------------------------------------------------------------------------
def active_rows(tok_state, flags):
    tok_state = np.asarray(tok_state)
    if flags & F_DCD:
        return np.flatnonzero(tok_state != TOK_CACHED)
    return np.arange(tok_state.shape[0])


# ----------------------------------------------------------------------------
# Sec. 4.1, second paragraph / Table 3 -- periodic refresh: every N-th step all
# tokens are recomputed, i.e. cached tokens count as newly accepted on that step.
# ----------------------------------------------------------------------------
def is_refresh_step(cfg, step_index):
    return cfg.refresh_every > 0 and step_index % cfg.refresh_every == 0


def refreshed_states(cfg, tok_state, step_index):
    tok_state = np.array(tok_state, dtype=np.uint8)
    if is_refresh_step(cfg, step_index):
        tok_state[tok_state == TOK_CACHED] = TOK_NEW
    return tok_state


# ----------------------------------------------------------------------------
# o2 -- Algorithm 1 "Router": one score per expert, softmax over all experts.
# Returns the fp32-rounded logits (on which experts are chosen) and the fp64
# softmax of those rounded logits.
# ----------------------------------------------------------------------------
def router(x, w_router):
    x64 = np.asarray(x, dtype=np.float64)
    w64 = np.asarray(w_router, dtype=np.float64)
    logits32 = (x64 @ w64.T).astype(np.float32)
    z = logits32.astype(np.float64)
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    probs = e / e.sum(axis=1, keepdims=True)
    return logits32, probs


# ----------------------------------------------------------------------------
# o3/o4 -- Eq. 4: a masked token is hot if its last confidence exceeds tau_h or
# if it lies within L_h positions of a decoded token; otherwise it is cold.
# Algorithm 1 step 1 then routes newly accepted and hot tokens first.
# ----------------------------------------------------------------------------
def classify(cfg, tok_state, conf, pos, group, branch):
    tok_state = np.asarray(tok_state)
    conf = np.asarray(conf, dtype=np.float32)
    T = tok_state.shape[0]
    tau = np.float32(cfg.tau_hot)
    cls = np.zeros(T, dtype=np.uint8)
    for t in range(T):
        s = tok_state[t]
        if s == TOK_CACHED:
            cls[t] = CLS_SKIP if (cfg.flags & F_DCD) else CLS_FIRST
        elif s == TOK_NEW:
            cls[t] = CLS_FIRST
        else:  # masked
            if not (cfg.flags & F_LAC):
                cls[t] = CLS_FIRST
                continue
            decoded = [pos[u] for u in range(T)
                       if group[u] == group[t] and branch[u] == branch[t]
                       and tok_state[u] in (TOK_NEW, TOK_CACHED)]
            if cfg.prefix_decoded:
                decoded.append(-1)
            if cfg.hot_dist_inclusive:
                near = any(abs(int(pos[t]) - int(j)) <= cfg.L_hot for j in decoded)
            else:
                near = any(abs(int(pos[t]) - int(j)) < cfg.L_hot for j in decoded)
            hot = bool(conf[t] > tau) or near
            cls[t] = CLS_FIRST if hot else CLS_COLD
    # A group whose first round would be empty: all its masked rows become hot.
    for g in set(int(v) for v in group):
        rows = [t for t in range(T) if group[t] == g and cls[t] != CLS_SKIP]
        if rows and not any(cls[t] == CLS_FIRST for t in rows):
            for t in rows:
                cls[t] = CLS_FIRST
    return cls


# ----------------------------------------------------------------------------
# o5/o7 -- top-k of one row, optionally restricted to an allowed expert set.
# Order: score descending, ties to the lower expert id.  margin is the gap
# between the last expert taken and the best one left out (inf if none is left).
# ----------------------------------------------------------------------------
def topk_row(logits32_row, k, allowed=None):
    cand = range(len(logits32_row)) if allowed is None else sorted(allowed)
    order = sorted(cand, key=lambda e: (-float(logits32_row[e]), e))
    take = order[:k]
    if len(order) > k:
        margin = float(logits32_row[order[k - 1]]) - float(logits32_row[order[k]])
    else:
        margin = float("inf")
    return take, margin


def routing_weights(probs_row, idx, norm_topk):
    p = np.array([probs_row[e] for e in idx], dtype=np.float64)
    return p / p.sum() if norm_topk else p


# ----------------------------------------------------------------------------
# o1-o8 -- the whole selection: Algorithm 1 plus the dispatch tables.
# ----------------------------------------------------------------------------
def select_experts(cfg, logits32, probs, tok_state, conf, pos, group, branch):
    T = len(tok_state)
    E, k, ns = cfg.n_experts, cfg.top_k, cfg.n_shared
    n_words = (E + 63) // 64
    cls = classify(cfg, tok_state, conf, pos, group, branch)

    idx = np.full((T, k), -1, dtype=np.int32)
    w = np.zeros((T, k), dtype=np.float64)
    margin = np.full(T, np.inf, dtype=np.float64)

    # first round: newly accepted and hot rows choose among all experts
    necessary = {}                                   # group -> set E_A(g)
    for t in range(T):
        if cls[t] == CLS_FIRST:
            take, margin[t] = topk_row(logits32[t], k)
            idx[t] = take
            w[t] = routing_weights(probs[t], take, cfg.norm_topk)
            necessary.setdefault(int(group[t]), set()).update(take)

    # second round: cold rows choose among the necessary experts of their group
    for t in range(T):
        if cls[t] == CLS_COLD:
            take, margin[t] = topk_row(logits32[t], k, allowed=necessary[int(group[t])])
            idx[t] = take
            w[t] = routing_weights(probs[t], take, cfg.norm_topk)

    group_mask = np.zeros((cfg.max_groups, n_words), dtype=np.uint64)
    for g, experts in necessary.items():
        for e in experts:
            group_mask[g, e // 64] |= np.uint64(1) << np.uint64(e % 64)

    # dispatch: slot id of (row t, choice j) is t*k+j; shared expert s of row t
    # is slot T*k + s*T + t and expert id E+s.  Slots are grouped by expert,
    # ascending slot id inside an expert.
    rows = [t for t in range(T) if cls[t] != CLS_SKIP]
    slots_of = [[] for _ in range(E + ns)]
    for t in rows:
        for j in range(k):
            slots_of[int(idx[t, j])].append(t * k + j)
    for s in range(ns):
        for t in rows:
            slots_of[E + s].append(T * k + s * T + t)
    cnt = np.array([len(v) for v in slots_of], dtype=np.int32)
    off = np.zeros(E + ns + 1, dtype=np.int32)
    off[1:] = np.cumsum(cnt)
    perm = np.full(T * (k + ns), -1, dtype=np.int32)
    flat = [s for v in slots_of for s in sorted(v)]
    perm[:len(flat)] = flat
    active = np.array([e for e in range(E + ns) if cnt[e] > 0], dtype=np.int32)

    return dict(tok_class=cls, topk_idx=idx, topk_w=w, margin=margin,
                group_mask=group_mask, expert_count=cnt, expert_offset=off,
                perm=perm, active=active, n_active=len(active),
                n_rows_active=len(rows))


def slot_row_weight(cfg, T, slot, topk_w):
    """Row and combine weight of a slot id (see select_experts)."""
    k = cfg.top_k
    if slot < T * k:
        return slot // k, float(topk_w[slot // k, slot % k])
    return (slot - T * k) % T, 1.0


# ----------------------------------------------------------------------------
# o9 -- one SwiGLU expert applied to a batch of rows: down(silu(gate x) * up x).
# ----------------------------------------------------------------------------
def expert_ffn(x_rows, w_gate_e, w_up_e, w_down_e):
    x64 = np.asarray(x_rows, dtype=np.float64)
    g = x64 @ np.asarray(w_gate_e, dtype=np.float64).T
    u = x64 @ np.asarray(w_up_e, dtype=np.float64).T
    a = g / (1.0 + np.exp(-g)) * u
    return a @ np.asarray(w_down_e, dtype=np.float64).T


# ----------------------------------------------------------------------------
# o1-o10 -- the whole layer step.  y_prev supplies the rows that are not
# recomputed (cached tokens keep the output of the step that last computed them).
# weights: dict with w_router [E,H], w_gate/w_up [E+ns,I,H], w_down [E+ns,H,I].
# ----------------------------------------------------------------------------
def moe_forward(cfg, weights, x, tok_state, conf, pos, group, branch, y_prev=None, step_index=0):
    tok_state = refreshed_states(cfg, tok_state, step_index)
    T = len(tok_state)
    logits32, probs = router(x, weights["w_router"])
    r = select_experts(cfg, logits32, probs, tok_state, conf, pos, group, branch)
    y = np.zeros((T, cfg.hidden), dtype=np.float64)
    if y_prev is not None:
        y[:] = np.asarray(y_prev, dtype=np.float64)
    for t in range(T):
        if r["tok_class"][t] != CLS_SKIP:
            y[t] = 0.0
    for e in r["active"]:
        slots = r["perm"][r["expert_offset"][e]:r["expert_offset"][e + 1]]
        rw = [slot_row_weight(cfg, T, int(s), r["topk_w"]) for s in slots]
        rows = [t for t, _ in rw]
        out = expert_ffn(np.asarray(x)[rows], weights["w_gate"][e],
                         weights["w_up"][e], weights["w_down"][e])
        for i, (t, wt) in enumerate(rw):
            y[t] += wt * out[i]
    r["logits"] = logits32
    r["probs"] = probs
    return y, r


# ----------------------------------------------------------------------------
# Stack glue for the MoE-only multi-layer workload: x <- x + y on computed
# rows (residual add), stored back in the activation type via round_fn.
# ----------------------------------------------------------------------------
def stack_forward(cfg, layers, x, tok_state, conf, pos, group, branch, round_fn=None):
    x = np.array(x, dtype=np.float64)
    n_act = []
    for weights in layers:
        y, r = moe_forward(cfg, weights, x, tok_state, conf, pos, group, branch)
        for t in range(len(tok_state)):
            if r["tok_class"][t] != CLS_SKIP:
                x[t] = x[t] + y[t]
        if round_fn is not None:
            x = round_fn(x)
        n_act.append(r["n_active"])
    return x, n_act
