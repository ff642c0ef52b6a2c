"""Thin Python binding over the C-ABI of libstairs_b200.so (see include/stairs.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch is used for device memory (weights, workspace, result buffers) and the stream.
There is no CPU fallback: loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstairs_b200.so")

STATUS = {0: "OK", 1: "EINVAL", 2: "ENOSPC", 3: "ESTATE", 4: "ECUDA", 5: "ETIMEOUT", 6: "EUNSUPPORTED"}

EXPORTS = ["stairs_workspace_bytes", "stairs_init", "stairs_prefill", "stairs_draft", "stairs_validate",
           "stairs_validate_host", "stairs_generate", "stairs_generate_adaptive", "stairs_sequence", "stairs_truncate", "stairs_sync",
           "stairs_launch_count", "stairs_profile", "stairs_profile_read", "stairs_reset",
           "stairs_destroy", "stairs_last_error", "stairs_accept_static", "stairs_debug_buffer", "stairs_debug_tune"]

STATIC_MAX_ROWS, STATIC_MAX_REQ = 1024, 64


class StairsError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"stairs: {STATUS.get(code, code)}: {text}")
        self.code = code


class CModel(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ff",
                                          "vocab", "max_pos", "norm", "act", "pos")] + \
               [("rope_theta", C.c_float), ("norm_eps", C.c_float), ("wdtype", C.c_int32)]


class CLayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("norm1_w", "norm1_b", "wq", "wk", "wv", "wo", "norm2_w", "norm2_b",
                                           "w_gate_or_fc1", "w_up", "w_down_or_fc2")]


class CWeights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("pos_emb", C.c_void_p), ("final_norm_w", C.c_void_p),
                ("final_norm_b", C.c_void_p), ("lm_head", C.c_void_p), ("layers", C.POINTER(CLayerW))]


class CConfig(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("target", CModel), ("draft", CModel),
                ("max_requests", C.c_int32), ("max_seq_len", C.c_int32), ("k_max", C.c_int32),
                ("kv_page_tokens", C.c_int32), ("kv_pages", C.c_int32), ("prefill_chunk", C.c_int32),
                ("device", C.c_int32), ("gemm_impl", C.c_int32), ("stream", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("wait_limit_cycles", C.c_uint64)]


class CStats(C.Structure):
    _fields_ = [("iterations", C.c_int32), ("drafted", C.c_int32), ("accepted", C.c_int32), ("emitted", C.c_int32),
                ("prefill_ms", C.c_float), ("draft_ms", C.c_float), ("validate_ms", C.c_float), ("total_ms", C.c_float)]


_lib = None


def load_library(path: Optional[str] = None):
    """dlopens the shared library and declares the signatures of include/stairs.h."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ImportError(f"{p} is missing: build it with `python -m paper_2407_19947_b200.build` "
                          "(there is no fallback implementation)")
    lib = C.CDLL(p)
    vp, i32p = C.c_void_p, C.POINTER(C.c_int32)
    lib.stairs_workspace_bytes.restype = C.c_size_t
    lib.stairs_workspace_bytes.argtypes = [C.POINTER(CConfig)]
    lib.stairs_init.argtypes = [C.POINTER(CConfig), C.POINTER(CWeights), C.POINTER(CWeights), C.POINTER(vp)]
    lib.stairs_prefill.argtypes = [vp, C.c_int, i32p, C.c_int]
    lib.stairs_draft.argtypes = [vp, C.c_int, C.c_int, vp]
    lib.stairs_validate.argtypes = [vp, C.c_int, i32p, i32p, vp, vp, vp, vp, C.c_int]
    lib.stairs_validate_host.argtypes = [vp, C.c_int, i32p, i32p, i32p, i32p, i32p, C.c_int]
    lib.stairs_generate.argtypes = [vp, C.c_int, i32p, C.c_int, C.c_int, C.c_int, C.c_int32, i32p, i32p,
                                    C.POINTER(CStats)]
    lib.stairs_generate_adaptive.argtypes = lib.stairs_generate.argtypes
    lib.stairs_sequence.argtypes = [vp, C.c_int, i32p, C.c_int, i32p]
    lib.stairs_truncate.argtypes = [vp, C.c_int, C.c_int]
    lib.stairs_sync.argtypes = [vp]
    lib.stairs_launch_count.restype = C.c_int64
    lib.stairs_launch_count.argtypes = [vp]
    lib.stairs_profile.argtypes = [vp, C.c_int]
    lib.stairs_profile_read.argtypes = [vp, C.POINTER(C.c_float), i32p, C.POINTER(C.c_float)]
    lib.stairs_reset.argtypes = [vp, C.c_int]
    lib.stairs_debug_buffer.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(C.c_size_t)]
    lib.stairs_debug_tune.argtypes = [vp, C.c_int, C.c_longlong]
    lib.stairs_destroy.argtypes = [vp]
    lib.stairs_accept_static.argtypes = [vp, C.c_int, C.c_int, C.c_int, i32p, vp, C.c_int, vp, vp, vp]
    lib.stairs_last_error.restype = C.c_char_p
    lib.stairs_last_error.argtypes = [vp]
    for name in EXPORTS:
        getattr(lib, name)  # raises AttributeError if the library lacks a declared symbol
    if path is None:
        _lib = lib
    return lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def c_model(shape) -> CModel:
    return CModel(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff,
                  shape.vocab, shape.max_pos, shape.norm, shape.act, shape.pos, shape.rope_theta, shape.norm_eps,
                  shape.wdtype)


class DeviceWeights:
    """Uploads one model's tensors (from a workloads.WeightSource) and keeps them alive."""

    def __init__(self, source, device: str):
        self.source, self.device = source, device
        shape = source.shape
        self.tensors = []

        def dev(layer, name):
            t = source.torch_tensor(layer, name, device)
            if t is None:
                return None
            self.tensors.append(t)
            return t.data_ptr()

        self.layers = (CLayerW * max(shape.n_layers, 1))()
        for l in range(shape.n_layers):
            for name, _ in CLayerW._fields_:
                setattr(self.layers[l], name, dev(l, name))
        self.c = CWeights(dev(-1, "tok_emb"), dev(-1, "pos_emb"), dev(-1, "final_norm_w"),
                          dev(-1, "final_norm_b"), dev(-1, "lm_head"),
                          C.cast(self.layers, C.POINTER(CLayerW)))


class Stairs:
    """One library context: a target model, an optional draft model, request slots."""

    def __init__(self, target_source, draft_source=None, *, max_requests=1, max_seq_len=512, k_max=8,
                 kv_page_tokens=64, kv_pages=0, prefill_chunk=0, device_index=0, gemm_impl=0, stream=None,
                 wait_limit_cycles=0):
        import torch
        self.torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("stairs needs a CUDA device (B200, sm_100a); there is no CPU path")
        self.device = f"cuda:{device_index}"
        torch.cuda.set_device(device_index)
        self.k_max, self.max_requests = k_max, max_requests
        self.vocab = target_source.shape.vocab
        self.tw = DeviceWeights(target_source, self.device)
        self.dw = DeviceWeights(draft_source, self.device) if draft_source is not None else None
        cfg = CConfig()
        cfg.struct_size = C.sizeof(CConfig)
        cfg.target = c_model(target_source.shape)
        if draft_source is not None:
            cfg.draft = c_model(draft_source.shape)
        cfg.max_requests, cfg.max_seq_len, cfg.k_max = max_requests, max_seq_len, k_max
        cfg.kv_page_tokens, cfg.kv_pages, cfg.prefill_chunk = kv_page_tokens, kv_pages, prefill_chunk
        cfg.device, cfg.gemm_impl = device_index, gemm_impl
        cfg.wait_limit_cycles = int(wait_limit_cycles)   # 0: the library's default bound for device-side waits
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        cfg.stream = self.stream.cuda_stream
        need = self.lib.stairs_workspace_bytes(C.byref(cfg))
        if need == 0:
            raise StairsError(1, self.lib.stairs_last_error(None).decode())
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace, cfg.workspace_bytes = base, need
        self.workspace_bytes = need
        self.cfg = cfg
        handle = C.c_void_p()
        rc = self.lib.stairs_init(C.byref(cfg), C.byref(self.tw.c), C.byref(self.dw.c) if self.dw else None,
                                  C.byref(handle))
        if rc:
            raise StairsError(rc, self.lib.stairs_last_error(None).decode())
        self.h = handle

    # -- helpers ----------------------------------------------------------------------------
    def _ck(self, rc: int):
        if rc:
            raise StairsError(rc, self.lib.stairs_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.lib.stairs_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C-ABI calls, same names ----------------------------------------------------------
    def prefill(self, req: int, prompt: Sequence[int]):
        p = _i32(prompt)
        self._ck(self.lib.stairs_prefill(self.h, req, _ptr(p), len(p)))

    def draft(self, req: int, k: int, draft_dev=None):
        """Returns the int32 device tensor holding the k drafted tokens."""
        if draft_dev is None:
            draft_dev = self.torch.zeros(max(self.k_max, 1), dtype=self.torch.int32, device=self.device)
        self._ck(self.lib.stairs_draft(self.h, req, k, draft_dev.data_ptr()))
        return draft_dev

    def validate(self, req_ids: Sequence[int], k: Sequence[int], draft_dev, *, commit=False, want_logits=False,
                 out=None):
        """Enqueues one stairs pass.  Returns (target_tokens_dev [n,k_max+1], accept_len_dev [n], logits or None)."""
        t = self.torch
        r, kk = _i32(req_ids), _i32(k)
        n = len(r)
        if out is None:
            tt = t.zeros((n, self.k_max + 1), dtype=t.int32, device=self.device)
            al = t.zeros((n,), dtype=t.int32, device=self.device)
        else:
            tt, al = out
        rows = int(kk.sum()) + n
        logits = t.empty((rows, self.vocab), dtype=t.float32, device=self.device) if want_logits else None
        self._ck(self.lib.stairs_validate(self.h, n, _ptr(r), _ptr(kk),
                                          draft_dev.data_ptr() if draft_dev is not None else None,
                                          tt.data_ptr(), al.data_ptr(),
                                          logits.data_ptr() if logits is not None else None, int(commit)))
        return tt, al, logits

    def validate_host(self, req_ids, k, draft_host, *, commit=False):
        """Host-buffer variant: (target_tokens [n,k_max+1], accept_len [n]) as numpy arrays."""
        r, kk = _i32(req_ids), _i32(k)
        n = len(r)
        d = _i32(draft_host).reshape(n, -1) if draft_host is not None and self.k_max > 0 else None
        if d is not None and d.shape[1] != self.k_max:
            pad = np.zeros((n, self.k_max), np.int32)
            pad[:, : d.shape[1]] = d
            d = pad
        tt = np.zeros((n, self.k_max + 1), np.int32)
        al = np.zeros((n,), np.int32)
        self._ck(self.lib.stairs_validate_host(self.h, n, _ptr(r), _ptr(kk), _ptr(d) if d is not None else None,
                                               _ptr(tt), _ptr(al), int(commit)))
        return tt, al

    def generate(self, req: int, prompt: Sequence[int], k: int, max_new: int, eos: int = -1, adaptive: bool = False):
        """Returns (new_tokens list, stats dict).  adaptive: stairs_generate_adaptive, k is the first draft length."""
        p = _i32(prompt)
        out = np.zeros(max(max_new, 1), np.int32)
        n_out = C.c_int32(0)
        st = CStats()
        fn = self.lib.stairs_generate_adaptive if adaptive else self.lib.stairs_generate
        self._ck(fn(self.h, req, _ptr(p), len(p), k, max_new, eos, _ptr(out), C.byref(n_out), C.byref(st)))
        stats = {n: getattr(st, n) for n, _ in CStats._fields_}
        return [int(x) for x in out[: n_out.value]], stats

    def sequence(self, req: int) -> List[int]:
        cap = self.cfg.max_seq_len
        buf = np.zeros(cap, np.int32)
        n = C.c_int32(0)
        self._ck(self.lib.stairs_sequence(self.h, req, _ptr(buf), cap, C.byref(n)))
        return [int(x) for x in buf[: n.value]]

    def truncate(self, req: int, n_tokens: int):
        self._ck(self.lib.stairs_truncate(self.h, req, n_tokens))

    def sync(self):
        self._ck(self.lib.stairs_sync(self.h))

    def launch_count(self) -> int:
        return int(self.lib.stairs_launch_count(self.h))

    def profile(self, enable: bool):
        self._ck(self.lib.stairs_profile(self.h, int(enable)))

    def profile_read(self):
        """(gemm_ms, gemm_launches, call_ms) of the most recent validate call."""
        g, n, c = C.c_float(0), C.c_int32(0), C.c_float(0)
        self._ck(self.lib.stairs_profile_read(self.h, C.byref(g), C.byref(n), C.byref(c)))
        return g.value, n.value, c.value

    def debug_buffer(self, which: int, dtype, count: int):
        """Copy of the first `count` elements of an internal activation buffer (tests only)."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        self._ck(self.lib.stairs_debug_buffer(self.h, which, C.byref(ptr), C.byref(nbytes)))
        t = self.torch
        off = ptr.value - self.workspace.data_ptr()
        esz = t.empty(0, dtype=dtype).element_size()
        assert count * esz <= nbytes.value
        self.sync()
        return self.workspace[off: off + count * esz].view(dtype).clone()

    def debug_tune(self, what: int, value: int):
        """Unstable tuning knob (see include/stairs_debug.h)."""
        self._ck(self.lib.stairs_debug_tune(self.h, what, value))

    def reset(self, req: int):
        self._ck(self.lib.stairs_reset(self.h, req))


def accept_static(logits_dev, k: Sequence[int], draft_dev, k_max: int, *, vocab: Optional[int] = None, stream=None):
    """stairs_accept_static: greedy token per row and accept length per request from logits that
    are already on the device, without a context and without any allocation inside the library
    (for callers that may not allocate device memory; the output tensors below are allocated
    here, by the caller's own torch allocator).  logits_dev: fp32 [rows, ld] torch tensor;
    draft_dev: int32 [n_req, k_max].  Returns (target_tokens [n_req, k_max+1], accept_len [n_req])."""
    import torch
    lib = load_library()
    kk = _i32(k)
    n = len(kk)
    tt = torch.zeros((n, k_max + 1), dtype=torch.int32, device=logits_dev.device)
    al = torch.zeros((n,), dtype=torch.int32, device=logits_dev.device)
    st = stream if stream is not None else torch.cuda.current_stream()
    rc = lib.stairs_accept_static(logits_dev.data_ptr(), vocab or logits_dev.shape[1], logits_dev.stride(0), n, _ptr(kk),
                                  draft_dev.data_ptr() if draft_dev is not None else None, k_max,
                                  tt.data_ptr(), al.data_ptr(), st.cuda_stream)
    if rc:
        raise StairsError(rc, lib.stairs_last_error(None).decode())
    return tt, al
