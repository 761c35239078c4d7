"""CPU oracle for TEAM's decode-loop glue: threshold acceptance, speculative branches for hot tokens and
their chained verification.  TEST INFRASTRUCTURE ONLY (tests, smoke and the benchmark's CPU legs may import it;
the CUDA path shares no code with it).

What the paper fixes:

  * Eq. 2-3: one forward pass gives every masked position a predicted token and a confidence c_k; a position is
    accepted when c_k > tau (tau = 0.95 in Sec. 5.1), the others stay masked.
  * Sec. 4.2 / Sec. 5.4: besides the base branch, three extra branches are built by additionally accepting the
    masked token with the highest confidence, the one with the second highest, and both (four branches, Sec. 5.1),
    "even when their confidence scores do not exceed the acceptance threshold"; the branches are decoded in the same
    forward pass and verified, and the aligned combinations {1st}, {2nd}, {1st + 2nd} allow verification in a chain.
  * Sec. 4.1: a token accepted at one step is computed once more at the next step and served from cache afterwards.

What it leaves open, and the reading taken here (plain Python loops; state per sequence):

  * Verification.  The base branch's results are always kept.  A speculated token is CONFIRMED in a branch when that
    branch's forward pass predicts the same token at its position with c > tau.  If the 1st candidate is confirmed
    in the base branch, the results of branch 1 (base + 1st) are trusted as well; if the 2nd candidate is then
    confirmed in branch 1, so are those of branch 3 (base + both).  If the 1st is not confirmed in the base branch
    but the 2nd is, branch 2 is trusted, and branch 3 after it if the 1st is confirmed in branch 2.  This is the
    chain; the last trusted branch is the ADOPTED one.
  * Acceptance.  Every masked position whose confidence exceeds tau in a trusted branch is accepted, with the
    prediction of the first trusted branch (in chain order) that accepts it; a confirmed candidate is accepted with
    its speculated token.  Hence: nothing confirmed => exactly the base branch's acceptance (Eq. 3).
  * A token accepted at this step is NEW at the next one (whichever branch accepted it), CACHED after that.
  * The next candidates are the two masked positions with the highest confidences in the adopted branch (ties to
    the lower position), their speculated tokens that branch's predictions.  Fewer than two masked positions left:
    fewer candidates (-1).
  * Rows of the next forward pass, ordered [sequence][branch][position]: branch 0 carries the base states, branch 1
    marks the 1st candidate NEW, branch 2 the 2nd, branch 3 both (a branch whose candidate does not exist repeats
    the base states).  The confidence handed to Eq. 4 is the adopted branch's for masked positions, 1 for decoded.
"""
import numpy as np

TOK_MASKED, TOK_NEW, TOK_CACHED = 0, 1, 2
N_BRANCHES = 4


def accept(conf_row, masked, tau):
    """Eq. 3: the masked positions whose confidence exceeds tau."""
    return [p for p in range(len(conf_row)) if masked[p] and np.float32(conf_row[p]) > np.float32(tau)]


def confirmed(pred_b, conf_b, pos, tok, tau):
    """A speculated (position, token) is confirmed by a branch's forward pass."""
    return pos >= 0 and int(pred_b[pos]) == int(tok) and np.float32(conf_b[pos]) > np.float32(tau)


def verify_chain(pred, conf, spec_pos, spec_tok, tau):
    """Sec. 5.4: which branches are trusted, in chain order.  pred, conf: [4][L] of one sequence."""
    chain = [0]
    if confirmed(pred[0], conf[0], spec_pos[0], spec_tok[0], tau):
        chain.append(1)
        if confirmed(pred[1], conf[1], spec_pos[1], spec_tok[1], tau):
            chain.append(3)
    elif confirmed(pred[0], conf[0], spec_pos[1], spec_tok[1], tau):
        chain.append(2)
        if confirmed(pred[2], conf[2], spec_pos[0], spec_tok[0], tau):
            chain.append(3)
    return chain


def branch_speculated(b, spec_pos):
    """Positions that branch b treats as already accepted on top of the base branch."""
    out = []
    if b in (1, 3) and spec_pos[0] >= 0:
        out.append(0)
    if b in (2, 3) and spec_pos[1] >= 0:
        out.append(1)
    return out


def build_branches(conf_row, masked):
    """Sec. 5.4: the two masked positions with the highest confidences (ties to the lower position)."""
    order = sorted((p for p in range(len(conf_row)) if masked[p]), key=lambda p: (-float(np.float32(conf_row[p])), p))
    return [order[0] if len(order) > 0 else -1, order[1] if len(order) > 1 else -1]


def seh_step(token, state, spec_pos, spec_tok, pred, conf, tau):
    """One decode step of one sequence.  token [L] (-1 while masked), state [L], spec_pos / spec_tok [2] describe
    the branches of the forward pass whose outputs pred / conf [4][L] are.  Returns the next token, state, spec_pos,
    spec_tok arrays, the adopted branch and the positions accepted at this step."""
    L = len(token)
    token, state = np.array(token, dtype=np.int32), np.array(state, dtype=np.uint8)
    chain = verify_chain(pred, conf, spec_pos, spec_tok, tau)
    newly = {}
    for b in chain:
        masked_b = [state[p] == TOK_MASKED for p in range(L)]
        for i in branch_speculated(b, spec_pos):
            p = int(spec_pos[i])
            masked_b[p] = False                       # decoded inside this branch ...
            newly.setdefault(p, int(spec_tok[i]))     # ... and confirmed, or the branch would not be trusted
        for p in accept(conf[b], masked_b, tau):
            newly.setdefault(p, int(pred[b][p]))
    adopted = chain[-1]
    for p in range(L):
        if state[p] == TOK_NEW:
            state[p] = TOK_CACHED
    for p, t in newly.items():
        token[p] = t
        state[p] = TOK_NEW
    masked = [state[p] == TOK_MASKED for p in range(L)]
    nxt = build_branches(conf[adopted], masked)
    nxt_tok = [int(pred[adopted][p]) if p >= 0 else -1 for p in nxt]
    return token, state, np.array(nxt, dtype=np.int32), np.array(nxt_tok, dtype=np.int32), adopted, sorted(newly)


def next_rows(state, spec_pos, conf_adopted, seq):
    """Rows of the next forward pass of one sequence: [branch][position] states, confidences, positions, group, branch."""
    L = len(state)
    rows = dict(tok_state=[], conf=[], pos=[], group=[], branch=[])
    for b in range(N_BRANCHES):
        st = np.array(state, dtype=np.uint8)
        for i in branch_speculated(b, spec_pos):
            st[int(spec_pos[i])] = TOK_NEW
        for p in range(L):
            rows["tok_state"].append(int(st[p]))
            rows["conf"].append(float(np.float32(conf_adopted[p])) if st[p] == TOK_MASKED else 1.0)
            rows["pos"].append(p)
            rows["group"].append(seq)
            rows["branch"].append(b)
    return rows


def decode_block(pred_steps, conf_steps, L, tau, max_steps=None, speculate=True):
    """Runs seh_step on one sequence until the block is fully decoded (or the script ends).  pred_steps / conf_steps:
    [steps][4][L].  speculate=False drops the branches (vanilla threshold decoding, Eq. 3 only).  Returns the
    per-step records and (forward passes, accepted tokens)."""
    token = np.full(L, -1, dtype=np.int32)
    state = np.zeros(L, dtype=np.uint8)
    spec_pos, spec_tok = np.array([-1, -1], dtype=np.int32), np.array([-1, -1], dtype=np.int32)
    records, forwards, accepted = [], 0, 0
    for s in range(len(pred_steps) if max_steps is None else min(max_steps, len(pred_steps))):
        if not (state == TOK_MASKED).any():
            break
        token, state, spec_pos, spec_tok, adopted, newly = seh_step(token, state, spec_pos, spec_tok, pred_steps[s],
                                                                   conf_steps[s], tau)
        if not speculate:
            spec_pos[:], spec_tok[:] = -1, -1
        forwards += 1
        accepted += len(newly)
        records.append(dict(token=token.copy(), state=state.copy(), spec_pos=spec_pos.copy(), spec_tok=spec_tok.copy(),
                            adopted=adopted, newly=newly))
    return records, forwards, accepted
