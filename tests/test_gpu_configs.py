"""GPU parity at the benchmark configs' own shapes (weights from the fast on-device generator; the
oracle receives device-to-host copies of the very same tensors).  Same bars as test_gpu_parity."""
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


def _rows_via_longest_row(tgt, prompt, draft):
    """Oracle logits of all stair rows from ONE forward of the longest row (row r's logits are the
    longest row's logits at position len(prompt)+r-1; the oracle's causality pin covers this),
    plus an independent forward of row 0 as a cross-check."""
    full = list(prompt) + [int(t) for t in draft]
    lg = so.forward_logits(tgt, full, all_positions=True)
    rows = lg[len(prompt) - 1: len(prompt) + len(draft)]
    row0 = so.forward_logits(tgt, list(prompt))
    assert np.abs(row0 - rows[0]).max() < 1e-3
    return rows


def test_config2_full_depth_rows_match_oracle():
    st = _stairs()
    w = wl.workload(2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=129))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=192, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    cont, _ = eng.generate(0, prompt, 0, 9)          # the library's own greedy continuation
    eng.prefill(0, prompt)
    draft = wl.forced_draft(np.array(cont), 5, w.target.vocab, 3)
    tt, al, logits = eng.validate([0], [8], torch.from_numpy(draft).cuda(), want_logits=True)
    eng.sync()
    ref = _rows_via_longest_row(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    err, exact = gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    # the forced draft agrees with the oracle's greedy tokens wherever the oracle is decisive
    oracle_tok = [so.argmax_lowest(r) for r in ref]
    for r in range(5):
        if so.top2_margin(ref[r]) >= gu.MARGIN:
            assert int(draft[r]) == oracle_tok[r]
    eng.close()


def test_config2_full_prefix_forced_accept_lengths_and_greedy_identity():
    st = _stairs()
    w = wl.workload(2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    prompt = wl.prompt_tokens(w, n=2049)
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=2064, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    cont = []
    for _ in range(9):
        t_host, _ = eng.validate_host([0], [0], None, commit=True)
        cont.append(int(t_host[0, 0]))
    eng.truncate(0, len(prompt))
    for k in (2, 4, 8):
        for i, a in enumerate(wl.forced_accept_lengths(k, 5, 40 + k)):
            d = np.zeros((1, 8), np.int32)
            d[0, :k] = wl.forced_draft(np.array(cont[: k + 1]), a, w.target.vocab, 7 + i)
            tt, al = eng.validate_host([0], [k], d)
            assert int(al[0]) == a and tt[0, : a + 1].tolist() == cont[: a + 1]
    # stairs generation with the 1-layer early-exit draft equals plain greedy on the same kernels
    short = prompt[:400]
    g0, _ = eng.generate(0, short, 0, 24)
    g4, s4 = eng.generate(0, short, 4, 24)
    assert g0 == g4 and s4["emitted"] >= 24
    eng.close()


@pytest.mark.parametrize("cfg,layers,draft_layers,n_prompt,k", [(3, 2, 1, 97, 4), (4, 2, 2, 301, 8)],
                         ids=["cfg3_shape_2layers", "cfg4_shape_2layers"])
def test_large_shapes_reduced_depth_match_oracle(cfg, layers, draft_layers, n_prompt, k):
    st = _stairs()
    w = _cut(wl.workload(cfg), layers, draft_layers)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=n_prompt))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=n_prompt + 64, k_max=8, kv_page_tokens=64)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, k)
    eng.sync()
    draft = d_dev.cpu().numpy()[:k]
    tt, al, logits = eng.validate([0], [k], d_dev, want_logits=True)
    eng.sync()
    ref = _rows_via_longest_row(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    g0, _ = eng.generate(0, prompt, 0, 20)
    gk, sk = eng.generate(0, prompt, k, 20)
    assert g0 == gk
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


def test_four_requests_of_different_lengths_in_one_call():
    # config-5 pattern at reduced depth and length: 4 requests, each its own k = 8 stair (36 rows)
    st = _stairs()
    w = _cut(wl.workload(5), 2, 2)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    lens = [700, 300, 1000, 520]
    eng = st.Stairs(tsrc, dsrc, max_requests=4, max_seq_len=1100, k_max=8, kv_page_tokens=64)
    prompts = [list(wl.prompt_tokens(w, request=i, n=n)) for i, n in enumerate(lens)]
    for i, p in enumerate(prompts):
        eng.prefill(i, p)
    rng = np.random.default_rng(9)
    drafts = rng.integers(0, w.target.vocab, size=(4, 8)).astype(np.int32)
    d_dev = torch.from_numpy(drafts).cuda()
    tt, al, logits = eng.validate([0, 1, 2, 3], [8, 8, 8, 8], d_dev, want_logits=True)
    eng.sync()
    logits = logits.cpu().numpy()
    for i in (1, 3):   # each request alone gives bit-identical rows
        tt1, al1, lg1 = eng.validate([i], [8], d_dev[i:i + 1].contiguous(), want_logits=True)
        eng.sync()
        np.testing.assert_array_equal(lg1.cpu().numpy(), logits[9 * i: 9 * i + 9])
        assert torch.equal(tt1[0], tt[i]) and int(al1[0]) == int(al[i])
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    ref = _rows_via_longest_row(tgt, prompts[1], drafts[1])
    gu.check_rows_against_oracle(logits[9:18], tt.cpu().numpy()[1], ref, gu.LOGIT_TOL_BF16)
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()


def test_sixty_four_rows_in_one_call():
    st = _stairs()
    shape = wl.family_b(2, 256, 8, 2, 64, 512, 2048, 512)
    tsrc = wl.WeightSource(shape, 7, "numpy", norm_jitter=0.1, std=0.03)
    tgt = so.OracleModel(shape, tsrc)
    prompt = list(wl.zipf_tokens(70, shape.vocab, 4))
    eng = st.Stairs(tsrc, None, max_requests=1, max_seq_len=160, k_max=63, kv_page_tokens=16)
    eng.prefill(0, prompt)
    cont = so.greedy_generate(tgt, prompt, 64)
    draft = wl.forced_draft(np.array(cont), 40, shape.vocab, 2)
    tt, al, logits = eng.validate([0], [63], torch.from_numpy(draft).cuda(), want_logits=True)
    eng.sync()
    ref = _rows_via_longest_row(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    eng.close()


def test_config4_full_depth_short_prompt_matches_oracle():
    st = _stairs()
    w = wl.workload(4)
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    prompt = list(wl.prompt_tokens(w, n=24))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=64, k_max=4, kv_page_tokens=64)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, 2)
    eng.sync()
    draft = d_dev.cpu().numpy()[:2]
    tt, al, logits = eng.validate([0], [2], d_dev, want_logits=True)
    eng.sync()
    tgt = so.OracleModel(w.target, tsrc, keep=False)     # one layer widened at a time (27 GB otherwise)
    full = prompt + [int(t) for t in draft]
    ref = so.forward_logits(tgt, full, all_positions=True)[len(prompt) - 1:]
    gpu_tok = tt.cpu().numpy()[0]
    err, exact = gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    print(f"7B full depth: logit max-abs err {err:.4f}, decisive rows {exact}/3")
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    eng.close()
    tsrc.drop_cache(); dsrc.drop_cache()
