"""GPU parity at the sizes the benchmark times (same bars as test_gpu_parity): the validation
microbench model at its full 2048-token prefix, the 3B- and 7B-shaped targets at their own prompt
lengths, one long-context request at the full 16384-token prefix, the attention path where one
unit walks several chunks, and the assistant's drafted tokens on the persistent-kernel path.

The oracle runs each check as ONE forward of the longest stair row: row r's logits are that
forward's logits at position len(prompt)+r-1 (the oracle's causality pin covers this); row 0 is
also computed on its own where that is cheap."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import stairs_oracle as so
from paper_2407_19947_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _stairs():
    from paper_2407_19947_b200 import build, stairs
    build.build()
    return stairs


def _cut(w, layers, draft_layers=1):
    return dataclasses.replace(w, target=w.target.replace(n_layers=layers), draft_layers=min(draft_layers, layers))


def _oracle_rows(tgt, prompt, draft, check_row0=True):
    full = [int(t) for t in prompt] + [int(t) for t in draft]
    x = so.forward_hidden(tgt, full)
    rows = so.logits_from_hidden(tgt, x[len(prompt) - 1:])
    if check_row0:
        row0 = so.forward_logits(tgt, [int(t) for t in prompt])
        assert np.abs(row0 - rows[0]).max() < 1e-3
    return rows


def _validate_and_compare(eng, tgt, prompt, draft, k, check_row0=True):
    d_dev = torch.zeros(max(eng.k_max, 1), dtype=torch.int32, device="cuda")
    d_dev[:k] = torch.from_numpy(np.asarray(draft[:k], np.int32))
    tt, al, logits = eng.validate([0], [k], d_dev, want_logits=True)
    eng.sync()
    ref = _oracle_rows(tgt, prompt, draft[:k], check_row0)
    gpu_tok = tt.cpu().numpy()[0]
    err, exact = gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft[:k], gpu_tok)
    return err, exact, ref, gpu_tok


def _own_continuation(eng, prompt, n):
    """The library's greedy continuation (n plain k = 0 steps), rolled back afterwards."""
    cont = []
    for _ in range(n):
        t_host, _ = eng.validate_host([0], [0], None, commit=True)
        cont.append(int(t_host[0, 0]))
    eng.truncate(0, len(prompt))
    return cont


def test_config2_full_depth_at_the_benchmarked_prefix():
    # the headline workload: 24 layers, 2048 cached tokens, k = 8 (nine stair rows)
    st = _stairs()
    w = wl.workload(2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=2049))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=2064, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    cont = _own_continuation(eng, prompt, 9)
    draft = wl.forced_draft(np.array(cont), 6, w.target.vocab, 3)
    err, exact, ref, gpu_tok = _validate_and_compare(eng, tgt, prompt, draft, 8)
    print(f"config 2, prefix 2048: logit max-abs err {err:.4f}, decisive rows {exact}/9")
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


@pytest.mark.parametrize("layers,n_prompt,k", [(32, 40, 4), (4, 513, 4)], ids=["full_depth_short", "4layers_p512"])
def test_config3_shape_matches_oracle(layers, n_prompt, k):
    st = _stairs()
    w = _cut(wl.workload(3), layers, 4)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=layers <= 4)
    prompt = list(wl.prompt_tokens(w, n=n_prompt))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=n_prompt + 64, k_max=4, kv_page_tokens=64)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, k)
    eng.sync()
    draft = d_dev.cpu().numpy()[:k]
    err, exact, _, _ = _validate_and_compare(eng, tgt, prompt, draft, k, check_row0=layers <= 4)
    print(f"config 3 shape, {layers} layers, prompt {n_prompt}: logit max-abs err {err:.4f}, decisive rows {exact}/{k + 1}")
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


def test_config4_shape_long_prompt_single_request_slot():
    # one request slot, k_max 8, a prompt past 448 tokens: the 64-row prefill passes need more
    # attention units than any validate call of this context
    st = _stairs()
    w = _cut(wl.workload(4), 2, 2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=1025))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=1025 + 64, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, 8)
    eng.sync()
    draft = d_dev.cpu().numpy()[:8]
    err, exact, _, _ = _validate_and_compare(eng, tgt, prompt, draft, 8)
    print(f"config 4 shape, 2 layers, prompt 1025: logit max-abs err {err:.4f}, decisive rows {exact}/9")
    g0, _ = eng.generate(0, prompt, 0, 12)
    g8, s8 = eng.generate(0, prompt, 8, 12)
    assert g0 == g8
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


def test_config4_full_depth_at_the_benchmarked_prompt():
    # all k+1 rows of three consecutive stairs iterations at the full 32 layers and the 1024-token
    # prompt: each call's drafts are forced from the library's own continuation (a different accept
    # length every time), the call commits, and the oracle recomputes the rows from the committed context
    st = _stairs()
    w = wl.workload(4)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    prompt = list(wl.prompt_tokens(w, n=1025))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=1025 + 64, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    tgt = so.OracleModel(w.target, tsrc, keep=False)     # one layer widened at a time
    ctx = list(prompt)
    for it, (k, a) in enumerate(((8, 4), (5, 5), (8, 0))):
        cont = _own_continuation(eng, ctx, k + 1)
        draft = wl.forced_draft(np.array(cont), a, w.target.vocab, 11 + it)
        d_dev = torch.zeros(8, dtype=torch.int32, device="cuda")
        d_dev[:k] = torch.from_numpy(draft)
        tt, al, logits = eng.validate([0], [k], d_dev, commit=True, want_logits=True)
        eng.sync()
        ref = _oracle_rows(tgt, ctx, draft, check_row0=False)
        gpu_tok = tt.cpu().numpy()[0]
        err, exact = gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
        acc = int(al.cpu()[0])
        assert acc == gu.first_mismatch(draft, gpu_tok) == a
        print(f"config 4, 32 layers, context {len(ctx)}, k {k}: logit max-abs err {err:.4f}, decisive rows {exact}/{k + 1}, accepted {acc}")
        new_ctx = eng.sequence(0)
        assert new_ctx == ctx + [int(t) for t in draft[:acc]] + [int(gpu_tok[acc])]
        ctx = new_ctx
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


def test_config5_one_request_at_the_full_prefix_two_layers():
    # 16384 cached tokens: 257 chunks per kv head, so every attention unit walks many chunks
    st = _stairs()
    w = _cut(wl.workload(5), 2, 2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=16385))
    eng = st.Stairs(tsrc, None, max_requests=1, max_seq_len=16384 + 64, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    draft = wl.uniform_tokens(8, w.target.vocab, 5)
    err, exact, _, _ = _validate_and_compare(eng, tgt, prompt, draft, 8, check_row0=False)
    print(f"config 5 shape, 2 layers, prefix 16384: logit max-abs err {err:.4f}, decisive rows {exact}/9")
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache()


@pytest.mark.parametrize("n_prompt", [1400, 2700, 5200], ids=str)
def test_units_that_walk_several_chunks(n_prompt):
    # eight kv heads and more than 18 chunks of 64 positions: heads x chunks exceeds the grid, so a
    # unit takes 2, 4 or 8 chunks in turn (the second chunk buffer is in use)
    st = _stairs()
    shape = wl.family_b(2, 512, 8, 8, 64, 1024, 2048, 8192)
    tsrc = wl.WeightSource(shape, 17, "numpy", norm_jitter=0.1, std=0.05)
    tgt = so.OracleModel(shape, tsrc)
    prompt = list(wl.zipf_tokens(n_prompt, shape.vocab, 23))
    eng = st.Stairs(tsrc, None, max_requests=1, max_seq_len=n_prompt + 64, k_max=8, kv_page_tokens=32)
    eng.prefill(0, prompt)
    cont = _own_continuation(eng, prompt, 9)
    draft = wl.forced_draft(np.array(cont), 5, shape.vocab, 9)
    _validate_and_compare(eng, tgt, prompt, draft, 8)
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()


def _check_drafted_tokens(drf, ctx, gpu_draft):
    """Teacher-forced on the library's own draft: token j must be the assistant's greedy token after
    ctx + draft[:j] wherever the oracle's top-2 margin is decisive, else within the margin."""
    decisive = 0
    for j, t in enumerate(gpu_draft):
        lg = so.forward_logits(drf, list(ctx) + [int(x) for x in gpu_draft[:j]])
        best = so.argmax_lowest(lg)
        if so.top2_margin(lg) >= gu.MARGIN:
            assert int(t) == best, f"drafted token {j}: {int(t)} != oracle {best}"
            decisive += 1
        else:
            assert lg[int(t)] >= lg[best] - gu.MARGIN
    return decisive


@pytest.mark.parametrize("early_exit", [True, False], ids=["early_exit_draft", "separate_draft"])
def test_drafted_tokens_match_the_oracle_assistant(early_exit):
    # the assistant's batch-1 loop on the persistent kernel: first step (two rows) and later steps
    st = _stairs()
    shape = wl.family_b(4, 256, 8, 2, 64, 512, 2048, 512)
    tsrc = wl.WeightSource(shape, 7, "numpy", norm_jitter=0.1, std=0.05)
    dshape = shape.replace(n_layers=2)
    if early_exit:
        dsrc = wl.WeightSource(dshape, 7, "numpy", norm_jitter=0.1, std=0.05, share_globals_with=tsrc, share_layers_with=tsrc)
    else:
        dsrc = wl.WeightSource(dshape, 99, "numpy", norm_jitter=0.1, std=0.05, share_globals_with=tsrc)
    drf = so.OracleModel(dshape, dsrc)
    prompt = list(wl.zipf_tokens(45, shape.vocab, 12))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=6, kv_page_tokens=16)
    launches = eng.launch_count()
    eng.prefill(0, prompt)
    # an early-exit assistant works on the main model's cache: the 44 prompt positions take one pass, not one per model
    assert eng.launch_count() - launches == (1 if early_exit else 2)
    decisive = 0
    for k in (1, 3, 6):
        d_dev = eng.draft(0, k)
        eng.sync()
        decisive += _check_drafted_tokens(drf, prompt, d_dev.cpu().numpy()[:k])
    # after committed validate calls (accept lengths the assistant does not know) the next drafts still follow
    for _ in range(4):
        d_dev = eng.draft(0, 4)
        eng.validate_host([0], [4], d_dev.cpu().numpy()[None, :4], commit=True)
        ctx = eng.sequence(0)
        d_dev = eng.draft(0, 3)
        eng.sync()
        decisive += _check_drafted_tokens(drf, ctx, d_dev.cpu().numpy()[:3])
    assert decisive >= 2     # random-init models are often undecided; the checks above hold either way
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()


def test_drafted_tokens_config4_shape_two_layer_draft():
    st = _stairs()
    w = _cut(wl.workload(4), 2, 2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    drf = so.OracleModel(w.draft, dsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=300))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=384, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, 4)
    eng.sync()
    _check_drafted_tokens(drf, prompt, d_dev.cpu().numpy()[:4])
    gu.assert_polled_scratch_empty(eng, "the calls of this test")
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()
