"""Pins for the attention oracle (in-block bidirectional attention over a KV cache with delayed insertion)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import attn_oracle as A


def _rows(S, B, L):
    pos = np.tile(np.arange(L), S * B)
    group = np.repeat(np.arange(S), B * L)
    branch = np.tile(np.repeat(np.arange(B), L), S)
    return pos, group, branch


def _inputs(rng, S, B, L, Hq, Hkv, d, P):
    T = S * B * L
    q = rng.standard_normal((T, Hq, d))
    k = rng.standard_normal((T, Hkv, d))
    v = rng.standard_normal((T, Hkv, d))
    kp = rng.standard_normal((S, P, Hkv, d))
    vp = rng.standard_normal((S, P, Hkv, d))
    kb = rng.standard_normal((S, L, Hkv, d))
    vb = rng.standard_normal((S, L, Hkv, d))
    return q, k, v, kp, vp, kb, vb


def test_full_recompute_equals_library_attention_over_prefix_and_block():
    """Delayed caching off: every row attends to its sequence's prefix and to the fresh keys of its own branch's
    block -- dense softmax attention, written here with torch's scaled_dot_product_attention (GQA by repetition)."""
    rng = np.random.default_rng(0)
    S, B, L, Hq, Hkv, d, P = 2, 2, 5, 4, 2, 8, 7
    q, k, v, kp, vp, kb, vb = _inputs(rng, S, B, L, Hq, Hkv, d, P)
    plen = np.array([7, 4])
    pos, group, branch = _rows(S, B, L)
    st = rng.integers(0, 3, S * B * L)
    out, _, _ = A.block_attention(q, k, v, kp, vp, plen, kb, vb, st, pos, group, branch, L, flags=0)
    for s in range(S):
        for b in range(B):
            rows = [t for t in range(S * B * L) if group[t] == s and branch[t] == b]
            K = np.concatenate([kp[s, :plen[s]], k[rows]], axis=0)              # [keys, Hkv, d]
            V = np.concatenate([vp[s, :plen[s]], v[rows]], axis=0)
            Kt = torch.from_numpy(np.repeat(K, Hq // Hkv, axis=1)).permute(1, 0, 2)   # [Hq, keys, d]
            Vt = torch.from_numpy(np.repeat(V, Hq // Hkv, axis=1)).permute(1, 0, 2)
            Qt = torch.from_numpy(q[rows]).permute(1, 0, 2)                     # [Hq, L, d]
            ref = F.scaled_dot_product_attention(Qt, Kt, Vt).permute(1, 0, 2).numpy()
            np.testing.assert_allclose(out[rows], ref, rtol=1e-10, atol=1e-12)


def test_cached_tokens_use_the_cache_and_get_no_output():
    """With delayed caching a cached token has no query (its output row is left alone) and the others see its CACHED
    key / value, not the fresh one: changing the fresh K/V of a cached row changes nothing, changing the cache does."""
    rng = np.random.default_rng(1)
    S, B, L, Hq, Hkv, d, P = 1, 1, 4, 2, 1, 4, 3
    q, k, v, kp, vp, kb, vb = _inputs(rng, S, B, L, Hq, Hkv, d, P)
    pos, group, branch = _rows(S, B, L)
    st = np.array([A.TOK_CACHED, A.TOK_NEW, A.TOK_MASKED, A.TOK_MASKED])
    prev = np.full((L, Hq, d), 9.0)
    out, ka, va = A.block_attention(q, k, v, kp, vp, [3], kb, vb, st, pos, group, branch, L, A.F_DCD, out_prev=prev)
    assert (out[0] == 9.0).all()
    k2, v2 = k.copy(), v.copy()
    k2[0] += 5.0
    v2[0] -= 3.0
    out2, _, _ = A.block_attention(q, k2, v2, kp, vp, [3], kb, vb, st, pos, group, branch, L, A.F_DCD, out_prev=prev)
    np.testing.assert_array_equal(out, out2)
    kb2 = kb.copy()
    kb2[0, 0] += 1.0
    out3, _, _ = A.block_attention(q, k, v, kp, vp, [3], kb2, vb, st, pos, group, branch, L, A.F_DCD, out_prev=prev)
    assert np.abs(out3[1:] - out[1:]).max() > 1e-6
    # insertion: only the newly accepted token (position 1) enters the cache
    np.testing.assert_array_equal(ka[0, 1], k[1])
    np.testing.assert_array_equal(va[0, 1], v[1])
    for p in (0, 2, 3):
        np.testing.assert_array_equal(ka[0, p], kb[0, p])


def test_delayed_caching_is_exact_when_decoded_tokens_are_stable():
    """Sec. 4.1's premise: once a decoded token has been through one more pass its representation is stable.  If the
    K/V of decoded tokens do not change after that pass, attention with delayed caching over a whole schedule equals
    recomputing every token at every step."""
    rng = np.random.default_rng(2)
    S, B, L, Hq, Hkv, d, P = 1, 1, 4, 2, 2, 4, 2
    pos, group, branch = _rows(S, B, L)
    kp, vp = rng.standard_normal((S, P, Hkv, d)), rng.standard_normal((S, P, Hkv, d))
    kb, vb = np.zeros((S, L, Hkv, d)), np.zeros((S, L, Hkv, d))
    frozen_k, frozen_v = rng.standard_normal((L, Hkv, d)), rng.standard_normal((L, Hkv, d))
    for step in range(6):
        st = np.array([A.TOK_NEW if step == p + 1 else (A.TOK_CACHED if step > p + 1 else A.TOK_MASKED) for p in range(L)])
        q = rng.standard_normal((L, Hq, d))
        k, v = rng.standard_normal((L, Hkv, d)), rng.standard_normal((L, Hkv, d))
        dec = st != A.TOK_MASKED
        k[dec], v[dec] = frozen_k[dec], frozen_v[dec]          # decoded tokens: the same K/V at every later pass
        full, _, _ = A.block_attention(q, k, v, kp, vp, [P], kb, vb, st, pos, group, branch, L, 0)
        dcd, kb, vb = A.block_attention(q, k, v, kp, vp, [P], kb, vb, st, pos, group, branch, L, A.F_DCD, out_prev=full)
        comp = st != A.TOK_CACHED
        np.testing.assert_allclose(dcd[comp], full[comp], rtol=1e-12, atol=1e-13)


def test_speculative_branches_are_isolated_and_do_not_write_the_cache():
    rng = np.random.default_rng(3)
    S, B, L, Hq, Hkv, d, P = 1, 2, 3, 2, 1, 4, 2
    q, k, v, kp, vp, kb, vb = _inputs(rng, S, B, L, Hq, Hkv, d, P)
    pos, group, branch = _rows(S, B, L)
    st = np.array([A.TOK_NEW, A.TOK_MASKED, A.TOK_MASKED,        # base branch
                   A.TOK_NEW, A.TOK_NEW, A.TOK_MASKED])          # branch 1 speculates position 1
    out, ka, va = A.block_attention(q, k, v, kp, vp, [2], kb, vb, st, pos, group, branch, L, A.F_DCD)
    k2 = k.copy()
    k2[3:] += 1.0                                                # branch 1's keys
    out2, _, _ = A.block_attention(q, k2, v, kp, vp, [2], kb, vb, st, pos, group, branch, L, A.F_DCD)
    np.testing.assert_array_equal(out[:3], out2[:3])             # the base branch does not see them
    np.testing.assert_array_equal(ka[0, 0], k[0])                # base NEW token inserted
    np.testing.assert_array_equal(ka[0, 1], kb[0, 1])            # the speculated one is not


def test_one_key_and_uniform_scores():
    """Closed forms: a single key returns its value; equal scores return the mean of the values."""
    d = 4
    q = np.ones((1, 1, d))
    k = np.zeros((1, 1, d))
    v = np.arange(d, dtype=float).reshape(1, 1, d)
    out, _, _ = A.block_attention(q, k, v, np.zeros((1, 0, 1, d)), np.zeros((1, 0, 1, d)), [0], np.zeros((1, 1, 1, d)),
                                  np.zeros((1, 1, 1, d)), [A.TOK_MASKED], [0], [0], [0], 1, 0)
    np.testing.assert_allclose(out[0, 0], v[0, 0])
    vp = np.stack([np.full(d, 2.0), np.full(d, 4.0)]).reshape(1, 2, 1, d)
    out, _, _ = A.block_attention(q, k, np.full((1, 1, d), 6.0), np.zeros((1, 2, 1, d)), vp, [2], np.zeros((1, 1, 1, d)),
                                  np.zeros((1, 1, 1, d)), [A.TOK_MASKED], [0], [0], [0], 1, 0)
    np.testing.assert_allclose(out[0, 0], np.full(d, 4.0))
