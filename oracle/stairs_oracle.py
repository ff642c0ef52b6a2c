"""CPU oracle for "stairs" assisted greedy generation.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the GPU library must compute.  It
may be imported by the tests, by the smoke check and by the benchmark's CPU
baseline leg, and by nothing else; it shares no code with the CUDA path and
imports nothing from it.  Inputs (weights, prompts, drafts) are handed in as
plain numpy arrays by the caller.

What it follows (paper section / figure):

* Section 3.1, Fig. 1: a model maps the tokens so far to a score for every
  vocabulary entry and the greedy choice is the highest-scoring entry
  (`forward_logits`, `greedy_token`).
* Section 3.1, Fig. 2: stand-alone greedy generation repeats that step
  (`greedy_generate`).
* Section 3.3, Fig. 4: the assistant drafts tokens; the drafted text is cut
  into sub-sequences that each contain one more token than the previous one,
  stacked in that order, and the main model predicts one further token for
  each (`stairs_rows`, `stairs_target_tokens`).
* Section 3.3, Fig. 5: the validation walk.  The first row (with its predicted
  token) is the ground truth; the next row is accepted only if, without its own
  last predicted token, it equals the ground truth, and then becomes the new
  ground truth; the walk ends at the first failure or the end of the batch and
  returns the ground truth (`stairs_validate_walk`).
* Section 3.2 ("such a cycle repeats"): the outer loop (`stairs_generate`).
* Section 3.2 and 4.1: the sequential assisted generation the paper compares with, one
  causal pass over context + draft and a dynamically set draft length
  (`assisted_generate`).

Precision: fp32 throughout (weights of bf16 models are the bf16 bit patterns
widened exactly to fp32).  Every stair row is an independent full causal
forward pass; there is no KV cache, no batching across rows, no blocking.

Readings where the paper is silent (architecture of the transformer itself,
tie-breaking): decoder-only pre-norm blocks of two families, see `forward_logits`;
argmax ties resolve to the lowest token id.

Pins (tests/test_oracle_*.py): the accept walk against a brute-force
first-mismatch search on exhaustive small cases; stairs output == stand-alone
greedy output for any draft and any k; k = 0 == greedy; family-A forward against
torch.nn.TransformerEncoderLayer; family-B forward against the HuggingFace Llama
implementation; closed-form special cases (uniform attention, position-shift
invariance of RoPE, causality); `assisted_generate` output == stand-alone greedy output
for any draft, and its draft-length schedule against closed forms (a perfect assistant: +2
per iteration up to the cap; an always-wrong one: down to 1, one token per iteration).
Acceptance-rate values are an empirical
property of random weights: parity unpinned, reported only.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

F32 = np.float32


# ----------------------------------------------------------------------------
# weights access
# ----------------------------------------------------------------------------
def widen(a: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> the exactly equal fp32 values; fp32 passes through."""
    if a is None:
        return None
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return np.ascontiguousarray(a, dtype=np.float32)


class OracleModel:
    """A model = a shape record (attributes n_layers, d_model, n_heads, n_kv_heads,
    head_dim, d_ff, vocab, norm, act, pos, rope_theta, norm_eps) plus a provider with
    `host_array(layer, name)`; layer -1 holds the global tensors.  Layers are widened
    on demand; `keep` bounds how many widened layers stay in memory."""

    def __init__(self, shape, provider, keep: bool = True):
        self.shape, self.provider, self.keep = shape, provider, keep
        self._mem = {}

    def w(self, layer: int, name: str):
        key = (layer, name)
        if key in self._mem:
            return self._mem[key]
        a = widen(self.provider.host_array(layer, name))
        if self.keep or layer < 0:
            self._mem[key] = a
        return a


# ----------------------------------------------------------------------------
# transformer pieces (fp32)
# ----------------------------------------------------------------------------
def layer_norm(x, g, b, eps):
    mu = x.mean(axis=-1, keepdims=True, dtype=F32)
    xc = x - mu
    var = (xc * xc).mean(axis=-1, keepdims=True, dtype=F32)
    return (xc / np.sqrt(var + F32(eps))) * g + b


def rms_norm(x, g, eps):
    ms = (x * x).mean(axis=-1, keepdims=True, dtype=F32)
    return (x / np.sqrt(ms + F32(eps))) * g


def gelu(x):
    """Exact (erf) form."""
    return (F32(0.5) * x * (F32(1.0) + _erf(x * F32(0.7071067811865476)))).astype(F32)


def silu(x):
    return (x / (F32(1.0) + np.exp(-x))).astype(F32)


def rope(u, positions, theta):
    """Rotary embedding on u[n, heads, hd]; element i pairs with i + hd/2; the pair is
    rotated by the angle position * theta^(-2i/hd)."""
    hd = u.shape[-1]
    half = hd // 2
    inv = (F32(theta) ** (-(np.arange(half, dtype=F32) * F32(2.0) / F32(hd)))).astype(F32)
    ang = positions.astype(F32)[:, None] * inv[None, :]            # [n, half]
    c, s = np.cos(ang).astype(F32)[:, None, :], np.sin(ang).astype(F32)[:, None, :]
    a, b = u[..., :half], u[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1).astype(F32)


def causal_attention(q, k, v, group):
    """q[n,Hq,hd], k/v[n,Hkv,hd]; query head h reads kv head h // group; position i sees
    positions 0..i.  Returns [n, Hq*hd]."""
    n, hq, hd = q.shape
    out = np.empty((n, hq, hd), dtype=F32)
    scale = F32(1.0 / np.sqrt(hd))
    mask = np.triu(np.ones((n, n), dtype=bool), 1)
    for h in range(hq):
        kh, vh = k[:, h // group, :], v[:, h // group, :]
        s = (q[:, h, :] @ kh.T) * scale
        s[mask] = -np.inf
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s, dtype=F32)
        p = p / p.sum(axis=-1, keepdims=True, dtype=F32)
        out[:, h, :] = p @ vh
    return out.reshape(n, hq * hd)


def forward_hidden(model: OracleModel, seq, n_layers=None, pos_offset: int = 0) -> np.ndarray:
    """Residual stream [n, d] after `n_layers` blocks (default: all), before the final norm.

    Family A (norm=0, act=0, pos=0): x = E[tok] + Epos[i]; per block
    x += Wo.attn(LN(x)); x += W2.gelu(W1.LN(x)).
    Family B (norm=1, act=1, pos=1): x = E[tok]; per block
    x += Wo.attn(rope(RMS(x))); x += Wd.(silu(Wg.h) * (Wu.h)), h = RMS(x).
    Weight matrices are [out, in]; there are no linear biases.  The first token sits at
    position `pos_offset` (0 in every use by the method; tests shift it)."""
    sh = model.shape
    seq = np.asarray(seq, dtype=np.int64)
    n = len(seq)
    positions = np.arange(n) + int(pos_offset)
    x = model.w(-1, "tok_emb")[seq].astype(F32)
    if sh.pos == 0:
        x = x + model.w(-1, "pos_emb")[positions]
    hq, hkv, hd = sh.n_heads, sh.n_kv_heads, sh.head_dim
    L = sh.n_layers if n_layers is None else n_layers
    for l in range(L):
        if sh.norm == 0:
            h = layer_norm(x, model.w(l, "norm1_w"), model.w(l, "norm1_b"), sh.norm_eps)
        else:
            h = rms_norm(x, model.w(l, "norm1_w"), sh.norm_eps)
        q = (h @ model.w(l, "wq").T).reshape(n, hq, hd)
        k = (h @ model.w(l, "wk").T).reshape(n, hkv, hd)
        v = (h @ model.w(l, "wv").T).reshape(n, hkv, hd)
        if sh.pos == 1:
            q, k = rope(q, positions, sh.rope_theta), rope(k, positions, sh.rope_theta)
        x = x + causal_attention(q, k, v, hq // hkv) @ model.w(l, "wo").T
        if sh.norm == 0:
            h = layer_norm(x, model.w(l, "norm2_w"), model.w(l, "norm2_b"), sh.norm_eps)
        else:
            h = rms_norm(x, model.w(l, "norm2_w"), sh.norm_eps)
        if sh.act == 0:
            x = x + gelu(h @ model.w(l, "w_gate_or_fc1").T) @ model.w(l, "w_down_or_fc2").T
        else:
            g = silu(h @ model.w(l, "w_gate_or_fc1").T)
            u = h @ model.w(l, "w_up").T
            x = x + (g * u) @ model.w(l, "w_down_or_fc2").T
        x = x.astype(F32)
    return x


def logits_from_hidden(model: OracleModel, x) -> np.ndarray:
    sh = model.shape
    if sh.norm == 0:
        h = layer_norm(x, model.w(-1, "final_norm_w"), model.w(-1, "final_norm_b"), sh.norm_eps)
    else:
        h = rms_norm(x, model.w(-1, "final_norm_w"), sh.norm_eps)
    return (h @ model.w(-1, "lm_head").T).astype(F32)


def forward_logits(model: OracleModel, seq, all_positions: bool = False) -> np.ndarray:
    """Vocabulary scores for the token following `seq` (Section 3.1): logits[V] of the last
    position, or [n, V] for every position when `all_positions`."""
    x = forward_hidden(model, seq)
    if all_positions:
        return logits_from_hidden(model, x)
    return logits_from_hidden(model, x[-1:])[0]


def argmax_lowest(logits) -> int:
    """Greedy choice; the lowest id wins a tie (np.argmax returns the first maximum)."""
    if not np.all(np.isfinite(logits)):
        raise FloatingPointError("non-finite logits")
    return int(np.argmax(logits))


def greedy_token(model: OracleModel, seq) -> int:
    return argmax_lowest(forward_logits(model, seq))


def top2_margin(logits) -> float:
    """Gap between the best and second-best score (used by the GPU parity rule)."""
    part = np.partition(logits, len(logits) - 2)
    return float(part[-1] - part[-2])


# ----------------------------------------------------------------------------
# stand-alone greedy (Section 3.1, Fig. 2)
# ----------------------------------------------------------------------------
def greedy_generate(model: OracleModel, prompt, max_new: int):
    seq = [int(t) for t in prompt]
    for _ in range(max_new):
        seq.append(greedy_token(model, seq))
    return seq[len(prompt):]


# ----------------------------------------------------------------------------
# one stairs iteration (Section 3.3)
# ----------------------------------------------------------------------------
def draft_tokens(draft_model: OracleModel, ctx, k: int):
    """The assistant's k greedy tokens after `ctx`."""
    seq = [int(t) for t in ctx]
    for _ in range(k):
        seq.append(greedy_token(draft_model, seq))
    return seq[len(ctx):]


def stairs_rows(ctx, draft):
    """Fig. 4: row r = ctx followed by the first r drafted tokens, r = 0..k, in order."""
    ctx = [int(t) for t in ctx]
    return [ctx + [int(t) for t in draft[:r]] for r in range(len(draft) + 1)]


def stairs_target_tokens(target_model: OracleModel, rows, with_margins: bool = False):
    """The main model's one additional token for each row; each row is its own forward."""
    toks, margins = [], []
    for row in rows:
        lg = forward_logits(target_model, row)
        toks.append(argmax_lowest(lg))
        margins.append(top2_margin(lg))
    return (toks, margins) if with_margins else toks


def stairs_validate_walk(rows, predicted):
    """Fig. 5.  rows[r] is the r-th sub-sequence, predicted[r] the main model's token for it.
    Returns (ground_truth, accept_len): ground_truth is the full accepted sequence and
    accept_len the number of rows after the first that were validated (= drafted tokens
    kept).  The ground truth starts as row 0 plus its predicted token; row r is validated
    if the row itself (i.e. without its predicted token) equals the current ground truth,
    and then row r plus its predicted token becomes the ground truth."""
    ground = list(rows[0]) + [int(predicted[0])]
    accepted = 0
    for r in range(1, len(rows)):
        if list(rows[r]) != ground:
            break
        ground = list(rows[r]) + [int(predicted[r])]
        accepted += 1
    return ground, accepted


def stairs_step(target_model: OracleModel, ctx, draft):
    """Rows, the target's token per row, and the walk.  Returns a dict with target_tokens
    (k+1), margins (k+1), accept_len and emitted (the accept_len+1 new tokens)."""
    rows = stairs_rows(ctx, draft)
    toks, margins = stairs_target_tokens(target_model, rows, with_margins=True)
    ground, a = stairs_validate_walk(rows, toks)
    return {"target_tokens": toks, "margins": margins, "accept_len": a,
            "emitted": ground[len(ctx):]}


# ----------------------------------------------------------------------------
# outer loop (Section 3.2 / 3.3)
# ----------------------------------------------------------------------------
def stairs_generate(target_model: OracleModel, draft_model, prompt, k: int, max_new: int,
                    draft_fn=None):
    """Repeat {draft k tokens, stairs rows, predict, validate, append} until max_new tokens.
    The draft length of an iteration is min(k, remaining - 1) so that nothing generated is
    thrown away.  `draft_fn(ctx, k)` may replace the assistant (tests use it to inject
    arbitrary drafts).  Returns (new_tokens, stats)."""
    ctx = [int(t) for t in prompt]
    out = []
    stats = {"iterations": 0, "drafted": 0, "accepted": 0}
    while len(out) < max_new:
        k_eff = min(k, max_new - len(out) - 1)
        if draft_fn is not None:
            d = [int(t) for t in draft_fn(ctx, k_eff)]
        else:
            d = draft_tokens(draft_model, ctx, k_eff)
        res = stairs_step(target_model, ctx, d)
        out.extend(res["emitted"])
        ctx.extend(res["emitted"])
        stats["iterations"] += 1
        stats["drafted"] += k_eff
        stats["accepted"] += res["accept_len"]
    return out[:max_new], stats


# ----------------------------------------------------------------------------
# sequential assisted generation with a dynamic draft length (Section 3.2, Section 4.1)
# ----------------------------------------------------------------------------
def assisted_generate(target_model: OracleModel, draft_model, prompt, k_first: int, k_max: int,
                      max_new: int, draft_fn=None):
    """The comparison method of the paper (Section 3.2): the assistant drafts, the main model
    processes the context plus the whole draft in ONE causal forward pass and its predictions
    are compared with the drafted tokens from left to right; the first main-model token that
    differs replaces the draft from there on.  The draft length is set dynamically
    (Section 4.1); the schedule taken here is the one of the library the paper uses: two more
    tokens after an iteration that kept every draft, one fewer (at least one) otherwise, never
    more than k_max.  Returns (new_tokens, stats); stats["k_schedule"] lists the draft lengths."""
    ctx = [int(t) for t in prompt]
    out = []
    stats = {"iterations": 0, "drafted": 0, "accepted": 0, "k_schedule": []}
    k_cur = int(k_first)
    while len(out) < max_new:
        k_eff = min(k_cur, max_new - len(out) - 1)
        if draft_fn is not None:
            d = [int(t) for t in draft_fn(ctx, k_eff)]
        else:
            d = draft_tokens(draft_model, ctx, k_eff)
        lg = forward_logits(target_model, ctx + d, all_positions=True)[len(ctx) - 1:]
        pred = [argmax_lowest(row) for row in lg]           # main model's token after ctx + d[:r], r = 0..k
        a = 0
        while a < k_eff and d[a] == pred[a]:
            a += 1
        emitted = d[:a] + [pred[a]]
        out.extend(emitted)
        ctx.extend(emitted)
        stats["iterations"] += 1
        stats["drafted"] += k_eff
        stats["accepted"] += a
        stats["k_schedule"].append(k_eff)
        if k_eff > 0:
            k_cur = min(k_cur + 2, k_max) if a == k_eff else max(1, k_cur - 1)
    return out[:max_new], stats
