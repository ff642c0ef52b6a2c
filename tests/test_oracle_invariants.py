"""Pins for the oracle's generation loops.

The method's claim (paper abstract, Sections 1 and 5) is a speed-up with no loss of
accuracy: the validation rule keeps a drafted token only when it is the main model's
own greedy token for the same context, so the generated text must be, token for
token, what the main model generates alone.  "Batch size 1" (k = 0) is stand-alone
generation (Section 4.3).
"""
import os

import numpy as np
import pytest

from oracle import stairs_oracle as so
from paper_2407_19947_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_pair(family="a"):
    if family == "a":
        shape = wl.family_a(3, 64, 4, 128, 211, 96, wl.WDTYPE_F32)
    else:
        shape = wl.family_b(3, 64, 4, 2, 16, 96, 211, 96, wl.WDTYPE_F32)
    src = wl.WeightSource(shape, 11, "numpy", norm_jitter=0.1, std=0.2)
    tgt = so.OracleModel(shape, src)
    dshape = shape.replace(n_layers=1)
    drf = so.OracleModel(dshape, wl.WeightSource(dshape, 11, "numpy", norm_jitter=0.1, std=0.2,
                                                 share_globals_with=src, share_layers_with=src))
    return tgt, drf


@pytest.mark.parametrize("family", ["a", "b"])
@pytest.mark.parametrize("k", [0, 1, 3, 6])
def test_stairs_output_equals_standalone_greedy(family, k):
    tgt, drf = small_pair(family)
    prompt = wl.uniform_tokens(9, tgt.shape.vocab, 1)
    ref = so.greedy_generate(tgt, prompt, 14)
    out, stats = so.stairs_generate(tgt, drf, prompt, k, 14)
    assert out == ref
    assert stats["iterations"] <= 14 and stats["accepted"] <= stats["drafted"]
    if k == 0:
        assert stats["iterations"] == 14 and stats["drafted"] == 0


def test_output_is_independent_of_the_draft():
    tgt, _ = small_pair("b")
    prompt = wl.uniform_tokens(7, tgt.shape.vocab, 2)
    ref = so.greedy_generate(tgt, prompt, 12)
    rng = np.random.default_rng(0)

    def random_draft(ctx, k):
        return rng.integers(0, tgt.shape.vocab, size=k)

    def perfect_draft(ctx, k):
        done = len(ctx) - len(prompt)
        return ref[done:done + k]

    def half_right(ctx, k):
        d = list(perfect_draft(ctx, k))
        if len(d) > 2:
            d[2] = (d[2] + 1) % tgt.shape.vocab
        return d

    out_r, st_r = so.stairs_generate(tgt, None, prompt, 4, 12, draft_fn=random_draft)
    out_p, st_p = so.stairs_generate(tgt, None, prompt, 4, 12, draft_fn=perfect_draft)
    out_h, st_h = so.stairs_generate(tgt, None, prompt, 4, 12, draft_fn=half_right)
    assert out_r == ref and out_p == ref and out_h == ref
    # a perfect draft is always fully accepted: k+1 tokens per iteration
    assert st_p["accepted"] == st_p["drafted"] and st_p["iterations"] == 3
    # the corrupted draft keeps exactly its first two tokens whenever it has more than two
    assert st_h["iterations"] == 4 and st_h["accepted"] == 2 + 2 + 2 + 2
    assert st_r["iterations"] >= st_h["iterations"]


def test_stairs_step_reports_target_tokens_for_every_row():
    tgt, drf = small_pair("a")
    ctx = list(wl.uniform_tokens(6, tgt.shape.vocab, 3))
    d = so.draft_tokens(drf, ctx, 3)
    res = so.stairs_step(tgt, ctx, d)
    assert len(res["target_tokens"]) == 4 and len(res["margins"]) == 4
    for r in range(4):
        assert res["target_tokens"][r] == so.greedy_token(tgt, ctx + d[:r])
    a = res["accept_len"]
    assert res["emitted"] == d[:a] + [res["target_tokens"][a]]


def test_config1_matches_committed_golden_tokens():
    # tests/golden/cfg1_greedy_tokens.txt is written by tests/golden/make_golden.py, which
    # calls only the oracle and the input generators.
    w = wl.workload(1)
    tsrc, dsrc = wl.make_sources(w)
    tgt, drf = so.OracleModel(w.target, tsrc), so.OracleModel(w.draft, dsrc)
    prompt = wl.prompt_tokens(w)
    with open(os.path.join(GOLDEN, "cfg1_greedy_tokens.txt")) as f:
        lines = [ln for ln in f.read().splitlines() if ln and not ln.startswith("#")]
    golden = [int(t) for t in lines[0].split()]
    assert len(golden) == w.max_new
    out, stats = so.stairs_generate(tgt, drf, prompt, w.k, w.max_new)
    assert out == golden
    assert so.greedy_generate(tgt, prompt, 8) == golden[:8]


@pytest.mark.parametrize("family", ["a", "b"])
def test_early_exit_assistant_hidden_states_are_the_main_models_first_layers(family):
    # An assistant made of the main model's first n layers sees, at every position, exactly the main
    # model's residual stream after n layers; by causality (pinned in test_oracle_forward) a
    # position's stream does not depend on later tokens either.  This is what lets such an assistant
    # work on the main model's K/V cache instead of keeping its own.
    tgt, drf = small_pair(family)
    seq = wl.uniform_tokens(13, tgt.shape.vocab, 5)
    n = drf.shape.n_layers
    np.testing.assert_array_equal(so.forward_hidden(drf, seq), so.forward_hidden(tgt, seq, n_layers=n))
    # (a shorter sequence takes other BLAS blocking: equal up to fp32 rounding, not bit for bit)
    np.testing.assert_allclose(so.forward_hidden(tgt, seq, n_layers=n)[:9], so.forward_hidden(tgt, seq[:9], n_layers=n),
                               rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("family", ["a", "b"])
def test_assisted_generation_equals_greedy_and_follows_its_schedule(family):
    # Section 3.2 / 4.1: one causal pass over context + draft, draft length set dynamically
    tgt, drf = small_pair(family)
    prompt = wl.uniform_tokens(8, tgt.shape.vocab, 2)
    ref = so.greedy_generate(tgt, prompt, 20)
    out, stats = so.assisted_generate(tgt, drf, prompt, 2, 6, 20)
    assert out == ref
    assert stats["drafted"] == sum(stats["k_schedule"]) and stats["accepted"] <= stats["drafted"]
    # a perfect assistant (the main model itself): every draft kept, so 2, 4, 6, ... tokens drafted
    # and k + 1 tokens emitted per iteration
    out_p, st_p = so.assisted_generate(tgt, tgt, prompt, 2, 6, 20)
    assert out_p == ref and st_p["accepted"] == st_p["drafted"]
    assert st_p["k_schedule"][:3] == [2, 4, 6] and st_p["iterations"] == 4     # 3 + 5 + 7 + the last 5 of 20
    # an assistant that is always wrong: the length decays to 1 and every iteration emits one token
    wrong = lambda ctx, k: [(ref[len(ctx) - len(prompt) + i] + 1) % tgt.shape.vocab for i in range(k)]
    out_w, st_w = so.assisted_generate(tgt, None, prompt, 3, 6, 20, draft_fn=wrong)
    assert out_w == ref and st_w["accepted"] == 0 and st_w["iterations"] == 20
    assert st_w["k_schedule"][:4] == [3, 2, 1, 1]
    # the causal pass gives the same predictions as the stairs rows computed one by one
    d = so.draft_tokens(drf, list(prompt), 4)
    rows = so.stairs_rows(prompt, d)
    one_by_one = so.stairs_target_tokens(tgt, rows)
    lg = so.forward_logits(tgt, list(prompt) + d, all_positions=True)[len(prompt) - 1:]
    assert [so.argmax_lowest(r) for r in lg] == one_by_one
