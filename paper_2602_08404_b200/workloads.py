"""Seeded synthetic workloads for the TEAM MoE-layer step.

This module only produces inputs: layer weights, the per-step hidden states of
a decoding block, and the scripted token-state schedule (which positions are
masked, newly accepted or cached at each denoising step).  It contains none of
the method's arithmetic (no routing, no classification, no expert math), so
both the CUDA binding's callers and the CPU oracle's callers may use it.

The shapes follow SDAR-30B-A3B (128 experts, 8 per token; Sec. 5.2 of the
paper) and a LLaDA2.0-mini-like layer; real checkpoints and benchmark prompts
are replaced by these generators.  The hidden-state statistics follow the
paper's observations: masked tokens of a block are highly similar (Table 4:
average pairwise cosine about 0.85), a token's hidden state changes most right
after it is accepted and is then stable (Sec. 3, temporal-spatial locality),
and tokens are accepted roughly left to right in clusters.
"""

from dataclasses import dataclass, replace

import numpy as np

TOK_MASKED, TOK_NEW, TOK_CACHED = 0, 1, 2


@dataclass(frozen=True)
class Shape:
    name: str
    hidden: int
    n_experts: int
    top_k: int
    inter: int
    n_shared: int
    dtype: str            # "f32" or "bf16" (x and expert weights; router is fp32)
    block: int            # tokens per decoding block
    n_steps: int          # denoising steps in the scripted schedule
    unmask_per_step: int  # tokens accepted per accepting step
    unmask_every: int     # an accepting step every this many steps
    L_hot: int
    tau_hot: float
    seqs: int = 1
    branches: int = 1
    seed: int = 0

    @property
    def rows(self):
        return self.seqs * self.branches * self.block


C1 = Shape("c1_tiny_f32", 256, 16, 2, 128, 0, "f32", 4, 8, 1, 2, 1, 0.7, seed=1)
C2 = Shape("c2_sdar_bf16", 2048, 128, 8, 768, 0, "bf16", 4, 4, 1, 1, 1, 0.7, seed=2)
C3 = Shape("c3_llada_bf16", 2048, 256, 8, 512, 1, "bf16", 32, 8, 4, 1, 3, 0.7, seed=3)


def c4(seqs):
    """Batch sweep on the SDAR shape: seqs sequences x 4 speculative branches x block 4."""
    return replace(C2, name=f"c4_sdar_b{seqs}", seqs=seqs, branches=4, seed=4 + seqs)


def paper_point():
    """The operating point of the paper's experiments (Sec. 5.1) on the SDAR shape: one sequence, block of 32
    tokens, 4 speculative branches (128 rows in one group), L_hot = 3, 4 tokens accepted per step."""
    return replace(C2, name="paper_block32_x4", block=32, branches=4, n_steps=8, unmask_per_step=4, L_hot=3, seed=17)


C5_LAYERS = 48
C5_BLOCKS = 64

# Small shapes that keep the structure of C2/C3 (ragged tails, several tiles)
# but let the oracle finish in well under a second; used by parity tests.
MINI_BF16 = Shape("mini_bf16", 256, 32, 4, 192, 0, "bf16", 8, 6, 1, 1, 1, 0.7, seed=11)
MINI_SHARED = Shape("mini_shared_bf16", 128, 24, 3, 64, 1, "bf16", 12, 5, 2, 1, 2, 0.7,
                    seqs=2, branches=2, seed=12)


# Enough k-blocks to wrap the expert kernel's smem ring inside one GEMM phase and enough work
# units that every CTA of a 148-SM grid processes several.
MINI_WRAP = Shape("mini_wrap_bf16", 768, 64, 4, 192, 0, "bf16", 16, 4, 3, 1, 2, 0.7,
                  seqs=2, branches=2, seed=13)


# Few rows, many activated experts with a wide intermediate dimension and a shared expert: in vanilla
# mode every CTA of a 148-SM grid gets more column groups than one pass of the few-rows expert kernel
# holds, so its range spans several passes and windows are shared between neighbouring CTAs.
STREAM_MULTI = Shape("stream_multi_bf16", 1024, 48, 8, 1024, 1, "bf16", 8, 4, 2, 1, 2, 0.7, seed=14)

# More rows than the few-rows kernel keeps resident: its gather mode (work items of 8 token-slots, several
# items for the experts that more than 8 rows chose), with a shared expert that every row uses.
STREAM_GATHER = Shape("stream_gather_bf16", 1024, 48, 8, 512, 1, "bf16", 12, 4, 3, 1, 2, 0.7, seqs=2, seed=15)

# Enough rows per call that the gather mode works on items of 16 token-slots (two token tiles per weight fragment).
STREAM_GATHER16 = Shape("stream_gather16_bf16", 1024, 48, 8, 512, 1, "bf16", 40, 4, 6, 1, 3, 0.7, seqs=2, seed=16)

# The limits of the resident mode: 8 rows x top-16 = 128 slots, 256 routed experts + 2 shared ones (a bit set
# of 258 bits), narrow experts (8 column groups each).
STREAM_WIDE = Shape("stream_k16_e256_bf16", 1024, 256, 16, 128, 2, "bf16", 8, 3, 2, 1, 2, 0.7, seed=18)

def round_to_bf16(a):
    """Round fp32 values to the nearest bf16-representable value (ties to even); returns fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def _store(shape, a):
    return round_to_bf16(a) if shape.dtype == "bf16" else np.ascontiguousarray(a, dtype=np.float32)


def make_weights(shape, seed=None, std=0.02):
    """Layer weights, N(0, std): router fp32 [E,H]; gate/up [E+ns,I,H]; down [E+ns,H,I].

    Returned as fp32 numpy arrays whose values are exactly representable in the
    shape's storage type.
    """
    rng = np.random.Generator(np.random.Philox(shape.seed * 1000 + 17 if seed is None else seed))
    E, H, I, ns = shape.n_experts, shape.hidden, shape.inter, shape.n_shared

    def normal(*dims):
        a = rng.standard_normal(dims, dtype=np.float32)
        a *= np.float32(std)
        return a

    return dict(
        w_router=normal(E, H),
        w_gate=_store(shape, normal(E + ns, I, H)),
        w_up=_store(shape, normal(E + ns, I, H)),
        w_down=_store(shape, normal(E + ns, H, I)),
    )


def device_layer_weights(shape, layer_seed, device, std=0.02):
    """One layer's weights generated ON THE DEVICE with torch's seeded generator (same distribution as
    make_weights): router fp32 [E,H]; gate/up [E+ns,I,H] and down [E+ns,H,I] (row-major) in the storage type.
    For workloads whose weights are too many to draw on the host (a 48-layer stack is 58 GB in bf16); a host-side
    consumer copies the tensors back, so both sides see the same values."""
    import torch
    E, H, I, ns = shape.n_experts, shape.hidden, shape.inter, shape.n_shared
    store = torch.bfloat16 if shape.dtype == "bf16" else torch.float32
    gen = torch.Generator(device=device)
    gen.manual_seed(int(layer_seed))
    wr = (torch.randn((E, H), generator=gen, device=device, dtype=torch.float32) * std).contiguous()
    wg, wu, wd = [(torch.randn(dims, generator=gen, device=device, dtype=torch.float32) * std).to(store).contiguous()
                  for dims in ((E + ns, I, H), (E + ns, I, H), (E + ns, H, I))]
    return wr, wg, wu, wd


def make_decode_script(n_seqs, block, n_steps, seed, n_branches=4, vocab=1000, rise=1.8, slope=0.5, boost=2.5):
    """Scripted outputs of a language-model head for a decode loop: pred int32 and conf fp32 [steps][S][branches][L].

    Stands in for the model's predictions (Eq. 2), which need a trained checkpoint.  The script does not depend on
    the decoding state: it gives every position a prediction and a confidence at every step, and the decode loop
    reads the ones it needs.  Confidence follows sigmoid(rise * (step + 1) - slope * position + boost * [branch has
    extra accepted tokens] + noise): it grows from step to step, falls from left to right (tokens are accepted in a
    near-autoregressive order, Sec. 3) and is a little higher in branches that carry speculated tokens.  The
    prediction is the sequence's fixed target token, except that an unconfident position sometimes predicts
    another token."""
    rng = np.random.Generator(np.random.Philox(seed))
    truth = rng.integers(0, vocab, size=(n_seqs, 1, block))
    steps = np.arange(n_steps).reshape(n_steps, 1, 1, 1)
    pos = np.arange(block).reshape(1, 1, 1, block)
    extra = np.array([0, 1, 1, 2][:n_branches], dtype=np.float64).reshape(1, 1, n_branches, 1)
    z = rise * (steps + 1) - slope * pos + boost * extra + rng.normal(0.0, 0.7, size=(n_steps, n_seqs, n_branches, block))
    conf = (1.0 / (1.0 + np.exp(-z))).astype(np.float32)
    other = rng.integers(0, vocab, size=conf.shape)
    wrong = rng.random(conf.shape) > 0.4 + 0.6 * conf
    pred = np.where(wrong, other, np.broadcast_to(truth[None], conf.shape)).astype(np.int32)
    return pred, conf


def _accept_step(shape, p):
    """Step at whose end position p is accepted (it is NEW at the following step)."""
    return (p // shape.unmask_per_step + 1) * shape.unmask_every - 1


def base_states(shape, step):
    """Token states of one sequence's base branch at a step (left-to-right acceptance)."""
    st = np.zeros(shape.block, dtype=np.uint8)
    for p in range(shape.block):
        a = _accept_step(shape, p)
        if step == a + 1:
            st[p] = TOK_NEW
        elif step > a + 1:
            st[p] = TOK_CACHED
    return st


def make_schedule(shape, seed=None, common=0.8, ar=0.8, branch_corr=0.95):
    """Scripted decoding of one block: a list of per-step input dicts.

    Each step gives x [T,H] (fp32 values exact in the storage type), tok_state
    u8[T], conf f32[T], pos/group/branch i32[T], with rows ordered
    [sequence][branch][position].

    Hidden states: a masked row is sqrt(common)*c + sqrt(1-common)*u_p, with c
    shared by the sequence and u_p an AR(1) process over positions (coefficient
    ar), which gives adjacent-position correlation common+(1-common)*ar and a
    floor of `common`.  From step to step h <- 0.9 h + 0.1 noise.  A row is
    redrawn independently when it becomes NEW and frozen afterwards.  Branch b>0
    additionally accepts the masked token(s) with the highest (b=1), second
    highest (b=2) or both (b=3) confidences; its other rows are branch_corr-
    correlated copies of the base rows.
    """
    rng = np.random.Generator(np.random.Philox(shape.seed * 1000 + 29 if seed is None else seed))
    H, L, S, B = shape.hidden, shape.block, shape.seqs, shape.branches

    def z(*dims):
        return rng.standard_normal(dims, dtype=np.float32)

    c = z(S, 1, H)
    u = np.empty((S, L, H), dtype=np.float32)
    u[:, 0] = z(S, H)
    for p in range(1, L):
        u[:, p] = ar * u[:, p - 1] + np.sqrt(1 - ar * ar) * z(S, H)
    h = np.sqrt(common) * c + np.sqrt(1 - common) * u          # [S, L, H] base branch
    steps = []
    for step in range(shape.n_steps):
        if step > 0:
            h = 0.9 * h + 0.1 * z(S, L, H)
        st0 = base_states(shape, step)
        for p in range(L):
            if st0[p] == TOK_NEW:
                h[:, p] = z(S, H)
        conf0 = rng.uniform(0.0, 0.95, size=(S, L)).astype(np.float32)
        x = np.empty((S, B, L, H), dtype=np.float32)
        state = np.empty((S, B, L), dtype=np.uint8)
        conf = np.empty((S, B, L), dtype=np.float32)
        for s in range(S):
            masked = [p for p in range(L) if st0[p] == TOK_MASKED]
            ranked = sorted(masked, key=lambda p: (-conf0[s, p], p))
            for b in range(B):
                extra = []
                if b in (1, 3) and len(ranked) > 0:
                    extra.append(ranked[0])
                if b in (2, 3) and len(ranked) > 1:
                    extra.append(ranked[1])
                stb = st0.copy()
                if b == 0:
                    xb = h[s].copy()
                else:
                    xb = branch_corr * h[s] + np.sqrt(1 - branch_corr ** 2) * z(L, H)
                    for p in range(L):
                        if st0[p] != TOK_MASKED:
                            xb[p] = h[s, p]
                for p in extra:
                    stb[p] = TOK_NEW
                    xb[p] = z(H)
                cb = conf0[s].copy()
                cb[stb != TOK_MASKED] = 1.0
                x[s, b], state[s, b], conf[s, b] = xb, stb, cb
        T = S * B * L
        pos = np.tile(np.arange(L, dtype=np.int32), S * B)
        group = np.repeat(np.arange(S, dtype=np.int32), B * L)
        branch = np.tile(np.repeat(np.arange(B, dtype=np.int32), L), S)
        steps.append(dict(x=_store(shape, x.reshape(T, H)), tok_state=state.reshape(T),
                          conf=conf.reshape(T), pos=pos, group=group, branch=branch))
    return steps
