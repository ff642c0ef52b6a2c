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
