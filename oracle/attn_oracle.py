"""CPU oracle for the attention half of delayed caching (Sec. 4.1; block diffusion, Sec. 2).
TEST INFRASTRUCTURE ONLY (tests, smoke and the benchmark's CPU legs may import it; the CUDA path shares no code
with it).

What the paper fixes:

  * Block diffusion (Sec. 2): attention is bidirectional inside the block that is being decoded and causal across
    blocks, so the keys and values of earlier blocks come from a KV cache (the "prefix").
  * Delayed caching (Sec. 4.1): at each iteration only the masked tokens and the tokens newly accepted in the
    previous step are computed; the key-value pairs of tokens decoded in earlier iterations are reused from cache;
    after each forward pass the KV pairs of the newly accepted tokens are inserted into the cache.

Reading taken where the paper is silent (plain loops, fp64 on exactly widened inputs):

  * One call = one attention layer of one denoising step.  Rows are ordered [sequence][branch][position]; every
    (sequence, branch) presents its whole block of L positions.  A row is COMPUTED unless delayed caching is on and
    its token is cached; only computed rows have a query and produce an output row, the others keep their output.
  * Keys / values seen by a computed row of (sequence s, branch b): the prefix of s (prefix_len[s] entries), then
    for every position p of the block the FRESH key / value of the row of (s, b) at p if that row is computed, else
    the entry p of the sequence's in-block cache.  All of them, masked positions included: attention inside the
    block is bidirectional.  Scores are q . k / sqrt(head_dim); softmax over all keys; grouped-query attention maps
    query head h to key/value head h // (n_heads // n_kv_heads).
  * Insertion after the pass: the fresh key / value of every computed row of the BASE branch (branch 0) whose token
    is decoded (newly accepted; or cached, when delayed caching is off and everything is recomputed) is written to
    the in-block cache at its position.  A token that only a speculative branch treats as accepted is not inserted:
    the cache is shared by the branches of a sequence.
"""
import numpy as np

TOK_MASKED, TOK_NEW, TOK_CACHED = 0, 1, 2
F_DCD = 1


def computed_rows(tok_state, flags):
    tok_state = np.asarray(tok_state)
    if flags & F_DCD:
        return tok_state != TOK_CACHED
    return np.ones(tok_state.shape[0], dtype=bool)


def block_attention(q, k_new, v_new, k_prefix, v_prefix, prefix_len, k_block, v_block, tok_state, pos, group, branch,
                    L, flags, out_prev=None):
    """q [T, Hq, d]; k_new, v_new [T, Hkv, d]; k_prefix, v_prefix [S, P, Hkv, d]; prefix_len [S];
    k_block, v_block [S, L, Hkv, d] (the in-block cache BEFORE the pass).  Returns (out [T, Hq, d], k_block', v_block')."""
    q, k_new, v_new = (np.asarray(a, dtype=np.float64) for a in (q, k_new, v_new))
    k_prefix, v_prefix = np.asarray(k_prefix, dtype=np.float64), np.asarray(v_prefix, dtype=np.float64)
    k_block, v_block = np.array(k_block, dtype=np.float64), np.array(v_block, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k_new.shape[1]
    rep = Hq // Hkv
    comp = computed_rows(tok_state, flags)
    out = np.zeros((T, Hq, d)) if out_prev is None else np.array(out_prev, dtype=np.float64)
    # the row of (sequence, branch) at position p
    row_at = {(int(group[t]), int(branch[t]), int(pos[t])): t for t in range(T)}
    for t in range(T):
        if not comp[t]:
            continue
        s, b = int(group[t]), int(branch[t])
        for h in range(Hq):
            g = h // rep
            keys = [k_prefix[s, j, g] for j in range(int(prefix_len[s]))]
            vals = [v_prefix[s, j, g] for j in range(int(prefix_len[s]))]
            for p in range(L):
                u = row_at[(s, b, p)]
                if comp[u]:
                    keys.append(k_new[u, g])
                    vals.append(v_new[u, g])
                else:
                    keys.append(k_block[s, p, g])
                    vals.append(v_block[s, p, g])
            scores = np.array([float(np.dot(q[t, h], kk)) for kk in keys]) / np.sqrt(d)
            w = np.exp(scores - scores.max())
            w /= w.sum()
            out[t, h] = sum(wi * vv for wi, vv in zip(w, vals))
    # delayed insertion: decoded tokens computed in the base branch enter the cache after the pass
    k_after, v_after = k_block.copy(), v_block.copy()
    for t in range(T):
        if comp[t] and int(branch[t]) == 0 and tok_state[t] in (TOK_NEW, TOK_CACHED):
            k_after[int(group[t]), int(pos[t])] = k_new[t]
            v_after[int(group[t]), int(pos[t])] = v_new[t]
    return out, k_after, v_after
