"""stairs_accept_static: the entry point for callers that cannot allocate device memory (code
running inside a pool that owns the device, or handed only finished buffers), so they have
neither a workspace nor a context.  Its scratch is a fixed array inside the library.  The
test feeds it the logits that stairs_validate dumped and expects exactly the tokens and accept
lengths stairs_validate itself returned (integers: the bar is equality), on two calls in a row
with different shapes, which also shows that stale keys from the first call are cleared."""
import numpy as np
import pytest
import torch

from paper_2407_19947_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_accept_matches_validate_on_two_calls_in_a_row():
    from paper_2407_19947_b200 import build, stairs
    build.build()
    shape = wl.family_b(2, 256, 8, 2, 64, 512, 4096, 256)
    src = wl.WeightSource(shape, 13, "numpy", norm_jitter=0.1, std=0.03)
    eng = stairs.Stairs(src, None, max_requests=2, max_seq_len=96, k_max=6, kv_page_tokens=16)
    eng.prefill(0, list(wl.zipf_tokens(30, shape.vocab, 1)))
    eng.prefill(1, list(wl.zipf_tokens(17, shape.vocab, 2)))
    rng = np.random.default_rng(0)
    for ks in ([6, 2], [0, 5]):
        # drafts that agree with the model for a while: take the model's own tokens, then corrupt one
        probe = torch.from_numpy(rng.integers(0, shape.vocab, size=(2, 6)).astype(np.int32)).cuda()
        tt0, _, _ = eng.validate([0, 1], ks, probe)
        eng.sync()
        drafts = probe.clone()
        drafts[0, 0] = tt0[0, 0]
        drafts[1, 0] = tt0[1, 0]
        tt, al, logits = eng.validate([0, 1], ks, drafts, want_logits=True)
        eng.sync()
        tt_s, al_s = stairs.accept_static(logits, ks, drafts, 6)
        torch.cuda.synchronize()
        for i, k in enumerate(ks):
            assert torch.equal(tt_s[i, : k + 1], tt[i, : k + 1])
        assert torch.equal(al_s, al)
        assert int(al[0]) >= (1 if ks[0] > 0 else 0)
    eng.close()


def test_static_accept_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2407_19947_b200 import build, stairs
    build.build()
    logits = torch.zeros((4, 128), dtype=torch.float32, device="cuda")
    drafts = torch.zeros((70, 63), dtype=torch.int32, device="cuda")
    # the checks run on the host before anything is launched, so undersized buffers are safe here
    with pytest.raises(stairs.StairsError) as e:
        stairs.accept_static(logits, [0] * (stairs.STATIC_MAX_REQ + 1), drafts, 63)
    assert e.value.code == 2 and "n_req" in str(e.value)
    with pytest.raises(stairs.StairsError) as e:
        stairs.accept_static(logits, [63] * 64, drafts, 63)            # 4096 rows > 1024
    assert e.value.code == 2 and "rows" in str(e.value)
    with pytest.raises(stairs.StairsError) as e:
        stairs.accept_static(logits, [5], drafts, 4)                   # k above k_max
    assert e.value.code == 1
