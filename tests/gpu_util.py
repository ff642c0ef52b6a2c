"""Helpers shared by the GPU parity tests (oracle on the host, library on the device)."""
import ctypes as C

import numpy as np

from oracle import stairs_oracle as so
from paper_2407_19947_b200 import workloads as wl

LOGIT_TOL_BF16 = 0.05   # max-abs logit error allowed for bf16 weights with fp32 accumulation
LOGIT_TOL_F32 = 1e-3    # fp32 weights
MARGIN = 0.1            # tokens must match bit-exactly where the oracle's top-2 margin is at least this


def oracle_pair(tsrc, dsrc=None, keep=True):
    tgt = so.OracleModel(tsrc.shape, tsrc, keep=keep)
    drf = so.OracleModel(dsrc.shape, dsrc, keep=keep) if dsrc is not None else None
    return tgt, drf


def oracle_stair_logits(tgt, ctx, draft):
    """Logits [k+1, V] of the stair rows, each row an independent full forward (no cache)."""
    rows = so.stairs_rows(ctx, draft)
    return np.stack([so.forward_logits(tgt, r) for r in rows]), rows


def first_mismatch(draft, target_tokens):
    for i, d in enumerate(draft):
        if int(d) != int(target_tokens[i]):
            return i
    return len(draft)


def check_rows_against_oracle(gpu_logits, gpu_tokens, oracle_logits, tol):
    """Element-wise logit bound, and token identity under the top-2 margin rule."""
    assert np.all(np.isfinite(gpu_logits))
    err = float(np.abs(gpu_logits - oracle_logits).max())
    assert err <= tol, f"logit max-abs error {err} > {tol}"
    exact = 0
    for r in range(oracle_logits.shape[0]):
        lg = oracle_logits[r]
        best = so.argmax_lowest(lg)
        if so.top2_margin(lg) >= MARGIN:
            assert int(gpu_tokens[r]) == best, f"row {r}: token {gpu_tokens[r]} != oracle {best}"
            exact += 1
        else:  # near-tie: the GPU's token must be within the margin of the oracle's best
            assert lg[int(gpu_tokens[r])] >= lg[best] - MARGIN
    return err, exact


def assert_polled_scratch_empty(eng, tag):
    """The persistent kernel's flagless hand-over buffers (split-tile sums, parked attention states):
    every word must read 0xffffffff ("empty") between calls."""
    import torch
    eng.sync()
    for which in (7, 8):
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        eng._ck(eng.lib.stairs_debug_buffer(eng.h, which, C.byref(ptr), C.byref(nbytes)))
        assert nbytes.value > 0
        words = eng.debug_buffer(which, torch.int32, nbytes.value // 4)
        bad = int((words != -1).sum())
        assert bad == 0, f"{bad} words of scratch {which} are not empty after {tag}"
