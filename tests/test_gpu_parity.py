"""GPU parity: the CUDA library (through its C-ABI) against the CPU oracle, on the same seeded
inputs.  Bars: fp32 weights - logits within 1e-3 and identical tokens; bf16 weights - logits
within max-abs 0.05 and tokens identical wherever the oracle's top-2 margin is >= 0.1; accept
lengths always equal the first mismatch recomputed from the library's own target tokens."""
import os

import numpy as np
import pytest
import torch

from oracle import stairs_oracle as so
from paper_2407_19947_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _stairs():
    from paper_2407_19947_b200 import build, stairs
    build.build()
    return stairs


def small_b(hq=8, hkv=2, hd=64, layers=3, d=256, f=512, v=2048, wdtype=wl.WDTYPE_BF16):
    return wl.family_b(layers, d, hq, hkv, hd, f, v, 512, wdtype)


def small_a(layers=3, d=256, heads=4, f=512, v=2048, wdtype=wl.WDTYPE_BF16):
    return wl.family_a(layers, d, heads, f, v, 512, wdtype)


def sources(shape, draft_layers=1, std=0.03, jitter=0.1, seed=7):
    tsrc = wl.WeightSource(shape, seed, "numpy", norm_jitter=jitter, std=std)
    dshape = shape.replace(n_layers=draft_layers)
    dsrc = wl.WeightSource(dshape, seed, "numpy", norm_jitter=jitter, std=std,
                           share_globals_with=tsrc, share_layers_with=tsrc)
    return tsrc, dsrc


# ---------------------------------------------------------------------------------------
# config 1: tiny fp32 model, whole generation
# ---------------------------------------------------------------------------------------
def test_config1_generation_equals_oracle_greedy_and_golden():
    st = _stairs()
    w = wl.workload(1)
    tsrc, dsrc = wl.make_sources(w)
    prompt = wl.prompt_tokens(w)
    with open(os.path.join(GOLDEN, "cfg1_greedy_tokens.txt")) as f:
        golden = [int(t) for t in [ln for ln in f.read().splitlines() if ln and not ln.startswith("#")][0].split()]
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=8, kv_page_tokens=16)
    out_k4, stats = eng.generate(0, prompt, w.k, w.max_new)
    out_k0, stats0 = eng.generate(0, prompt, 0, w.max_new)
    assert out_k0 == golden, "k=0 must be plain greedy"
    assert out_k4 == golden, "stairs output must equal stand-alone greedy"
    assert stats0["iterations"] == w.max_new and stats0["drafted"] == 0
    assert stats["iterations"] <= w.max_new and 0 <= stats["accepted"] <= stats["drafted"]
    assert stats["emitted"] == stats["iterations"] + stats["accepted"]
    # the oracle's stairs loop drafts with the same assistant: same iteration count
    tgt, drf = gu.oracle_pair(tsrc, dsrc)
    out_o, stats_o = so.stairs_generate(tgt, drf, prompt, w.k, w.max_new)
    assert out_o == golden
    assert stats_o["iterations"] == stats["iterations"] and stats_o["accepted"] == stats["accepted"]
    assert eng.sequence(0)[: len(prompt)] == [int(t) for t in prompt]
    eng.close()


def test_config1_validate_logits_match_oracle():
    st = _stairs()
    w = wl.workload(1)
    tsrc, dsrc = wl.make_sources(w)
    tgt, drf = gu.oracle_pair(tsrc, dsrc)
    prompt = list(wl.prompt_tokens(w))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=4, kv_page_tokens=16)
    eng.prefill(0, prompt)
    d_dev = eng.draft(0, 4)
    tt, al, logits = eng.validate([0], [4], d_dev, commit=False, want_logits=True)
    eng.sync()
    draft = d_dev.cpu().numpy()[:4].tolist()
    assert draft == so.draft_tokens(drf, prompt, 4)
    ref, _ = gu.oracle_stair_logits(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_F32)
    res = so.stairs_step(tgt, prompt, draft)
    assert gpu_tok[:5].tolist() == res["target_tokens"]
    assert int(al.cpu()[0]) == res["accept_len"] == gu.first_mismatch(draft, gpu_tok)
    eng.close()


# ---------------------------------------------------------------------------------------
# small bf16 models of both families: stair rows against the oracle
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [small_b(8, 2, 64), small_b(4, 4, 80, d=320, f=640), small_b(4, 1, 128, d=512),
                                   small_a()], ids=["gqa_hd64", "mha_hd80", "mqa_hd128", "family_a"])
@pytest.mark.parametrize("k", [0, 1, 4, 8])
@pytest.mark.parametrize("std", [0.03, 0.05], ids=["std0.03", "std0.05"])
def test_stair_rows_match_oracle_bf16(shape, k, std):
    # weight scale 0.03 gives these small models the logit scale of the benchmark configs (about
    # 0.7); 0.05 is the harder case for the absolute logit bar (logit scale about 2)
    st = _stairs()
    tsrc, dsrc = sources(shape, std=std)
    tgt, _ = gu.oracle_pair(tsrc)
    prompt = list(wl.zipf_tokens(37, shape.vocab, 21))          # crosses two 16-token pages, ragged tail
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=96, k_max=8, kv_page_tokens=16, prefill_chunk=16)
    eng.prefill(0, prompt)
    # the oracle's own greedy continuation, then a forced draft that matches its first a tokens
    cont = so.greedy_generate(tgt, prompt, k + 1)
    a = k // 2
    draft = wl.forced_draft(np.array(cont), a, shape.vocab, 5)
    d_dev = torch.zeros(8, dtype=torch.int32, device="cuda")
    d_dev[:k] = torch.from_numpy(draft)
    tt, al, logits = eng.validate([0], [k], d_dev, commit=False, want_logits=True)
    eng.sync()
    ref, _ = gu.oracle_stair_logits(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    assert 0 <= int(al.cpu()[0]) <= k
    eng.close()


def test_batched_requests_match_single_request_calls_bit_for_bit():
    st = _stairs()
    shape = small_b(8, 2, 64)
    tsrc, dsrc = sources(shape)
    eng = st.Stairs(tsrc, dsrc, max_requests=3, max_seq_len=128, k_max=8, kv_page_tokens=32)
    prompts = [list(wl.zipf_tokens(n, shape.vocab, 30 + i)) for i, n in enumerate((9, 40, 64))]
    ks = [8, 0, 3]
    for i, p in enumerate(prompts):
        eng.prefill(i, p)
    rng = np.random.default_rng(3)
    drafts = rng.integers(0, shape.vocab, size=(3, 8)).astype(np.int32)
    d_dev = torch.from_numpy(drafts).cuda()
    tt, al, logits = eng.validate([0, 1, 2], ks, d_dev, commit=False, want_logits=True)
    eng.sync()
    logits = logits.cpu().numpy()
    row = 0
    for i in range(3):
        tt1, al1, lg1 = eng.validate([i], [ks[i]], d_dev[i:i + 1].contiguous(), commit=False, want_logits=True)
        eng.sync()
        n = ks[i] + 1
        np.testing.assert_array_equal(lg1.cpu().numpy(), logits[row:row + n])
        np.testing.assert_array_equal(tt1.cpu().numpy()[0, :n], tt.cpu().numpy()[i, :n])
        assert int(al1.cpu()[0]) == int(al.cpu()[i])
        row += n
    # and the middle request against the oracle
    tgt, _ = gu.oracle_pair(tsrc)
    ref, _ = gu.oracle_stair_logits(tgt, prompts[2], drafts[2, :3])
    gu.check_rows_against_oracle(logits[10:14], tt.cpu().numpy()[2], ref, gu.LOGIT_TOL_BF16)
    eng.close()


@pytest.mark.parametrize("early_exit", [True, False])
def test_gpu_stairs_equals_gpu_greedy_token_for_token(early_exit):
    st = _stairs()
    shape = small_b(8, 2, 64, layers=4)
    tsrc, dsrc = sources(shape, draft_layers=2)
    if not early_exit:
        dshape = shape.replace(n_layers=2)
        dsrc = wl.WeightSource(dshape, 99, "numpy", norm_jitter=0.1, std=0.03, share_globals_with=tsrc)
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=160, k_max=6, kv_page_tokens=16)
    prompt = list(wl.zipf_tokens(50, shape.vocab, 8))
    ref, _ = eng.generate(0, prompt, 0, 64)
    for k in (1, 3, 6):
        out, stats = eng.generate(0, prompt, k, 64)
        assert out == ref, f"k={k}"
        assert stats["emitted"] >= 64 and stats["iterations"] <= 64
    eng.close()


def test_commit_appends_exactly_the_accepted_tokens():
    st = _stairs()
    shape = small_a()
    tsrc, dsrc = sources(shape)
    eng = st.Stairs(tsrc, dsrc, max_requests=2, max_seq_len=96, k_max=4, kv_page_tokens=16)
    prompt = list(wl.uniform_tokens(20, shape.vocab, 4))
    eng.prefill(1, prompt)
    # target's own continuation via k=0 calls without commit, then a draft that matches 2 tokens
    tt, al, _ = eng.validate([1], [0], None, commit=False)
    t0 = int(tt.cpu()[0, 0])
    tt_host, al_host = eng.validate_host([1], [0], None, commit=False)
    assert int(tt_host[0, 0]) == t0 and int(al_host[0]) == 0
    assert eng.sequence(1) == prompt, "commit=0 must not change the sequence"
    tt_host, al_host = eng.validate_host([1], [0], None, commit=True)
    assert eng.sequence(1) == prompt + [t0]
    # draft [x, y, z, w] where only the first matches
    nxt, _ = eng.validate_host([1], [0], None, commit=False)
    d = np.array([[int(nxt[0, 0]), 1, 2, 3]], np.int32)
    tt_host, al_host = eng.validate_host([1], [4], d, commit=False)
    a = gu.first_mismatch(d[0], tt_host[0])
    assert int(al_host[0]) == a >= 1
    tt2, al2 = eng.validate_host([1], [4], d, commit=True)
    np.testing.assert_array_equal(tt2, tt_host)
    assert eng.sequence(1) == prompt + [t0] + d[0, :a].tolist() + [int(tt_host[0, a])]
    eng.close()


def test_same_call_twice_is_bitwise_identical():
    st = _stairs()
    shape = small_b(4, 4, 80, d=320, f=640)
    tsrc, dsrc = sources(shape)
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=96, k_max=8, kv_page_tokens=16)
    eng.prefill(0, list(wl.zipf_tokens(33, shape.vocab, 2)))
    d_dev = torch.arange(8, dtype=torch.int32, device="cuda")
    a = eng.validate([0], [8], d_dev, commit=False, want_logits=True)
    b = eng.validate([0], [8], d_dev, commit=False, want_logits=True)
    eng.sync()
    assert torch.equal(a[2], b[2]) and torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    eng.close()


def test_error_paths_return_codes_and_leave_the_context_usable():
    st = _stairs()
    shape = small_a(layers=1)
    tsrc, dsrc = sources(shape)
    eng = st.Stairs(tsrc, dsrc, max_requests=2, max_seq_len=32, k_max=4, kv_page_tokens=16, kv_pages=3)
    d_dev = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(st.StairsError) as e:
        eng.validate([0], [2], d_dev)
    assert e.value.code == 3                       # ESTATE: not prefilled
    with pytest.raises(st.StairsError) as e:
        eng.prefill(5, [1, 2, 3])
    assert e.value.code == 1                       # EINVAL: slot out of range
    with pytest.raises(st.StairsError) as e:
        eng.prefill(0, [1])
    assert e.value.code == 1                       # EINVAL: prompt too short
    with pytest.raises(st.StairsError) as e:
        eng.prefill(0, [1, shape.vocab])
    assert e.value.code == 1                       # EINVAL: token out of range
    with pytest.raises(st.StairsError) as e:
        eng.prefill(0, list(range(40)))
    assert e.value.code == 2                       # ENOSPC: longer than max_seq_len
    eng.prefill(0, list(range(1, 30)))             # takes 2 of the 3 pages
    with pytest.raises(st.StairsError) as e:
        eng.prefill(1, list(range(1, 30)))
    assert e.value.code == 2                       # ENOSPC: pool exhausted
    with pytest.raises(st.StairsError) as e:
        eng.validate([0], [5], d_dev)
    assert e.value.code == 1                       # k > k_max
    with pytest.raises(st.StairsError) as e:
        eng.validate([0], [4], d_dev)
    assert e.value.code == 2                       # 29 + 5 > max_seq_len
    eng.reset(0)
    eng.prefill(1, list(range(1, 20)))
    tt, al = eng.validate_host([1], [2], np.array([[7, 8, 0, 0]], np.int32))
    assert 0 <= int(al[0]) <= 2
    eng.close()


@pytest.mark.parametrize("lengths", [[10], [17, 30], [65, 10], [33], [40, 10], [129]], ids=str)
def test_fresh_contexts_with_varied_call_shapes_complete(lengths):
    """Every row-box size as the very first launch of a context, then validate calls of several row
    counts and a draft: no device wait may run out (the sync would raise) and the library's own
    accept rule must hold for every request."""
    st = _stairs()
    shape = small_b()
    tsrc, dsrc = sources(shape)
    n = len(lengths)
    eng = st.Stairs(tsrc, dsrc, max_requests=n, max_seq_len=192, k_max=8, wait_limit_cycles=400000000)
    for r, length in enumerate(lengths):
        eng.prefill(r, list(wl.uniform_tokens(length, shape.vocab, 20 + r)))
    d = torch.from_numpy(wl.uniform_tokens(8 * n, shape.vocab, 31).reshape(n, 8).astype(np.int32)).cuda()
    for ks in ([8] * n, [0] * n, [3] * n):
        tt, al, _ = eng.validate(list(range(n)), ks, d)
        eng.sync()
        tt_h, al_h = tt.cpu().numpy(), al.cpu().numpy()
        for i in range(n):
            assert int(al_h[i]) == gu.first_mismatch(d[i, :ks[i]].cpu().numpy(), tt_h[i])
    eng.draft(0, 3)
    eng.sync()
    eng.close()


def test_expired_device_wait_is_reported_and_the_gpu_stays_usable():
    """Every wait inside the persistent kernel is bounded.  With the bound set to about a microsecond the
    waits of a healthy call run out: the kernel must drain and exit by itself, the next sync must
    report STAIRS_ETIMEOUT (5), and a context with the default bound must work afterwards."""
    st = _stairs()
    shape = small_b()
    tsrc, dsrc = sources(shape)
    prompt = list(wl.uniform_tokens(40, shape.vocab, 3))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=4, wait_limit_cycles=2000)
    with pytest.raises(st.StairsError) as e:
        eng.prefill(0, prompt)
        eng.sync()
    assert e.value.code == 5
    eng.close()
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=4)
    eng.prefill(0, prompt)
    tt, al = eng.validate_host([0], [2], np.array([[7, 8, 0, 0]], np.int32))
    assert 0 <= int(al[0]) <= 2
    eng.close()


@pytest.mark.parametrize("shape", [small_b(8, 2, 64), small_b(4, 4, 80, d=320, f=640), small_a()],
                         ids=["gqa_hd64", "mha_hd80", "family_a"])
def test_long_prefix_positions_split_over_several_units(shape):
    # 333 cached positions span six 64-position chunks, so the softmax of every row is assembled
    # from several units' partial states; pages of 32 tokens, ragged last page
    st = _stairs()
    shape = shape.replace(max_pos=512)
    tsrc, dsrc = sources(shape)
    tgt, _ = gu.oracle_pair(tsrc)
    prompt = list(wl.zipf_tokens(334, shape.vocab, 77))
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=400, k_max=8, kv_page_tokens=32, prefill_chunk=128)
    eng.prefill(0, prompt)
    k = 5
    cont = so.greedy_generate(tgt, prompt, k + 1)
    draft = wl.forced_draft(np.array(cont), 3, shape.vocab, 6)
    d_dev = torch.zeros(8, dtype=torch.int32, device="cuda")
    d_dev[:k] = torch.from_numpy(draft)
    tt, al, logits = eng.validate([0], [k], d_dev, commit=False, want_logits=True)
    eng.sync()
    ref, _ = gu.oracle_stair_logits(tgt, prompt, draft)
    gpu_tok = tt.cpu().numpy()[0]
    gu.check_rows_against_oracle(logits.cpu().numpy(), gpu_tok, ref, gu.LOGIT_TOL_BF16)
    assert int(al.cpu()[0]) == gu.first_mismatch(draft, gpu_tok)
    # the per-launch tensor-core path (other attention kernel, explicit norms) agrees closely
    eng2 = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=400, k_max=8, kv_page_tokens=32, prefill_chunk=128, gemm_impl=2)
    eng2.prefill(0, prompt)
    _, _, logits2 = eng2.validate([0], [k], d_dev, commit=False, want_logits=True)
    eng2.sync()
    assert float((logits2 - logits).abs().max()) < 0.03
    eng.close(); eng2.close()


def test_polled_scratch_is_empty_again_after_every_kind_of_call():
    # The persistent kernel hands split-tile sums and parked attention states over without flags:
    # a word reads 0xffffffff until it has been stored, and whoever read it puts the pattern back.
    # Whatever a call looked like (prefill passes of 64 rows, single draft rows, batched validate
    # calls with split contexts, a context switch to other shapes), every word must read "empty"
    # once the call is over - a leftover would be taken for a finished sum by a later call.
    st = _stairs()
    shape = small_b(8, 2, 64).replace(max_pos=512)
    tsrc, dsrc = sources(shape)
    eng = st.Stairs(tsrc, dsrc, max_requests=3, max_seq_len=400, k_max=8, kv_page_tokens=32)

    def all_empty(tag):
        gu.assert_polled_scratch_empty(eng, tag)

    all_empty("init")
    prompts = [list(wl.zipf_tokens(n, shape.vocab, 50 + i)) for i, n in enumerate((334, 70, 9))]
    for i, p in enumerate(prompts):
        eng.prefill(i, p)
        all_empty(f"prefill of {len(p)} tokens")
    d_dev = torch.from_numpy(np.random.default_rng(5).integers(0, shape.vocab, size=(3, 8)).astype(np.int32)).cuda()
    for ks in ([8, 3, 0], [0, 0, 0], [5, 8, 8]):
        eng.validate([0, 1, 2], ks, d_dev, commit=False)
        all_empty(f"validate {ks}")
    eng.validate([1], [4], d_dev[1:2].contiguous(), commit=True)
    all_empty("committing validate")
    eng.draft(0, 6)
    all_empty("draft")
    out, _ = eng.generate(2, prompts[2], 4, 12)
    all_empty("generate")
    assert len(out) == 12
    eng.close()


def test_adaptive_draft_length_generation_matches_the_oracle_schedule():
    # sequential assisted generation with a dynamic draft length (Sections 3.2 and 4.1): on the tiny
    # fp32 config the tokens are exact, so the library must walk the very schedule the oracle walks
    st = _stairs()
    w = wl.workload(1)
    tsrc, dsrc = wl.make_sources(w)
    prompt = wl.prompt_tokens(w)
    tgt, drf = gu.oracle_pair(tsrc, dsrc)
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=128, k_max=6, kv_page_tokens=16)
    out, stats = eng.generate(0, prompt, 2, 24, adaptive=True)
    ref, ref_stats = so.assisted_generate(tgt, drf, prompt, 2, 6, 24)
    assert out == ref == so.greedy_generate(tgt, prompt, 24)
    assert (stats["iterations"], stats["drafted"], stats["accepted"]) == (ref_stats["iterations"], ref_stats["drafted"], ref_stats["accepted"])
    with pytest.raises(st.StairsError) as e:
        eng.generate(0, prompt, 0, 8, adaptive=True)
    assert e.value.code == 1
    eng.close()
    # and on a bf16 model through the persistent kernel: same output as plain greedy on the same kernels
    shape = small_b(8, 2, 64, layers=4)
    tsrc, dsrc = sources(shape, draft_layers=2)
    eng = st.Stairs(tsrc, dsrc, max_requests=1, max_seq_len=160, k_max=6, kv_page_tokens=16)
    p2 = list(wl.zipf_tokens(50, shape.vocab, 8))
    g0, _ = eng.generate(0, p2, 0, 48)
    ga, sa = eng.generate(0, p2, 3, 48, adaptive=True)
    assert ga == g0 and sa["emitted"] >= 48 and sa["accepted"] <= sa["drafted"]
    eng.close()


@pytest.mark.parametrize("hq,hkv,hd", [(8, 2, 64), (4, 1, 128), (4, 4, 64)], ids=["gqa4_hd64", "mqa4_hd128", "mha_hd64"])
def test_tcgen05_attention_path_matches_oracle(hq, hkv, hd):
    # The attention contractions on the 5th-generation tensor cores are chosen per call for long
    # contexts and prefill passes; here they are switched on for every call, so that small models
    # reach them too: prefill passes of 64 rows (up to 256 queries per kv head: two query blocks),
    # contexts split over several units (partial states merged by the merge at the end of the attention phase) and not, two
    # requests in one call, several draft lengths.  Same bars as everywhere.
    st = _stairs()
    shape = wl.family_b(2, hq * hd if hq * hd <= 512 else 512, hq, hkv, hd, 512, 2048, 1024)
    tsrc, dsrc = sources(shape, std=0.05)
    tgt, _ = gu.oracle_pair(tsrc)
    eng = st.Stairs(tsrc, dsrc, max_requests=2, max_seq_len=700, k_max=8, kv_page_tokens=32)
    eng.debug_tune(3, 2)
    prompts = [list(wl.zipf_tokens(n, shape.vocab, 40 + i)) for i, n in enumerate((611, 75))]
    for i, p in enumerate(prompts):
        eng.prefill(i, p)
    for ks in ([8, 3], [0, 8], [1, 1]):
        drafts = np.zeros((2, 8), np.int32)
        for i in range(2):
            cont = so.greedy_generate(tgt, prompts[i], ks[i] + 1)
            drafts[i, :ks[i]] = wl.forced_draft(np.array(cont), ks[i] // 2, shape.vocab, 5 + i)
        tt, al, logits = eng.validate([0, 1], ks, torch.from_numpy(drafts).cuda(), commit=False, want_logits=True)
        eng.sync()
        logits = logits.cpu().numpy()
        row = 0
        for i in range(2):
            ref, _ = gu.oracle_stair_logits(tgt, prompts[i], drafts[i, :ks[i]])
            gpu_tok = tt.cpu().numpy()[i]
            gu.check_rows_against_oracle(logits[row:row + ks[i] + 1], gpu_tok, ref, gu.LOGIT_TOL_BF16)
            assert int(al.cpu()[i]) == gu.first_mismatch(drafts[i, :ks[i]], gpu_tok)
            row += ks[i] + 1
    # the same calls on the register path agree closely (different summation order only)
    _, _, lg_tc = eng.validate([0, 1], [8, 3], torch.from_numpy(drafts).cuda(), want_logits=True)
    eng.debug_tune(3, 1)
    _, _, lg_mma = eng.validate([0, 1], [8, 3], torch.from_numpy(drafts).cuda(), want_logits=True)
    eng.sync()
    assert float((lg_tc - lg_mma).abs().max()) < 5e-3
    gu.assert_polled_scratch_empty(eng, "tcgen05 attention calls")
    eng.close()
