"""Seeded synthetic inputs: model shapes, random-init weights, prompts, forced drafts.

This module only *generates data*.  It contains none of the method's arithmetic
(no transformer math, no argmax, no accept rule) and imports neither the CPU
oracle nor the CUDA binding; both of them consume the buffers produced here.

The paper evaluates trained T5 checkpoints on one natural-language prompt
(Section 4.1-4.2).  Neither is available offline, so random-init decoder-only
models of the benchmark configs' shapes and synthetic token ids stand in.

Weight recipe: every tensor is an independent stream keyed by
(seed, layer index, tensor index); values are 0.02 * standard normal; norm
gains are 1 and norm biases 0 (optionally jittered for tests, so that a path
that ignores a gain or bias is caught).  bf16 models round the fp32 draw to
bf16 once (round-to-nearest-even); both consumers receive those 16-bit
patterns.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np

NORM_LAYERNORM, NORM_RMSNORM = 0, 1
ACT_GELU, ACT_SWIGLU = 0, 1
POS_LEARNED, POS_ROPE = 0, 1
WDTYPE_F32, WDTYPE_BF16 = 0, 1

# per-layer tensor order (index = stream key)
LAYER_TENSORS = ("norm1_w", "norm1_b", "wq", "wk", "wv", "wo",
                 "norm2_w", "norm2_b", "w_gate_or_fc1", "w_up", "w_down_or_fc2")
GLOBAL_TENSORS = ("tok_emb", "pos_emb", "final_norm_w", "final_norm_b", "lm_head")


@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Architecture of one decoder-only transformer (field names follow the C header)."""
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    max_pos: int
    norm: int = NORM_RMSNORM
    act: int = ACT_SWIGLU
    pos: int = POS_ROPE
    rope_theta: float = 1.0e4
    norm_eps: float = 1.0e-5
    wdtype: int = WDTYPE_BF16

    def replace(self, **kw) -> "ModelShape":
        return dataclasses.replace(self, **kw)

    def tensor_shape(self, name: str):
        d, hq, hkv, hd, f, v = (self.d_model, self.n_heads, self.n_kv_heads,
                                self.head_dim, self.d_ff, self.vocab)
        return {
            "tok_emb": (v, d), "pos_emb": (self.max_pos, d), "lm_head": (v, d),
            "final_norm_w": (d,), "final_norm_b": (d,),
            "norm1_w": (d,), "norm1_b": (d,), "norm2_w": (d,), "norm2_b": (d,),
            "wq": (hq * hd, d), "wk": (hkv * hd, d), "wv": (hkv * hd, d),
            "wo": (d, hq * hd),
            "w_gate_or_fc1": (f, d), "w_up": (f, d), "w_down_or_fc2": (d, f),
        }[name]

    def has_tensor(self, name: str) -> bool:
        if name == "pos_emb":
            return self.pos == POS_LEARNED
        if name == "w_up":
            return self.act == ACT_SWIGLU
        if name.endswith("_b"):
            return self.norm == NORM_LAYERNORM
        return True

    def weight_bytes_per_call(self) -> int:
        """Bytes of weights one forward pass streams once (embedding rows excluded)."""
        es = 4 if self.wdtype == WDTYPE_F32 else 2
        per_layer = 0
        for n in ("wq", "wk", "wv", "wo", "w_gate_or_fc1", "w_up", "w_down_or_fc2"):
            if self.has_tensor(n):
                s = self.tensor_shape(n)
                per_layer += s[0] * s[1]
        return es * (per_layer * self.n_layers + self.vocab * self.d_model)

    def kv_bytes_per_token(self) -> int:
        es = 4 if self.wdtype == WDTYPE_F32 else 2
        return 2 * self.n_kv_heads * self.head_dim * es * self.n_layers


def family_a(n_layers, d_model, n_heads, d_ff, vocab, max_pos, wdtype) -> ModelShape:
    """Pre-LayerNorm, learned positions, MHA, 2-matrix GELU MLP (configs 1 and 2)."""
    return ModelShape(n_layers, d_model, n_heads, n_heads, d_model // n_heads, d_ff, vocab,
                      max_pos, NORM_LAYERNORM, ACT_GELU, POS_LEARNED, 1.0e4, 1.0e-5, wdtype)


def family_b(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, max_pos,
             wdtype=WDTYPE_BF16) -> ModelShape:
    """Pre-RMSNorm, RoPE (theta 1e4, rotate-half pairs), SwiGLU (configs 3-5)."""
    return ModelShape(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab,
                      max_pos, NORM_RMSNORM, ACT_SWIGLU, POS_ROPE, 1.0e4, 1.0e-5, wdtype)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark config: target/draft shapes and the generation recipe."""
    name: str
    target: ModelShape
    draft_layers: int            # number of draft layers
    draft_shares_target: bool    # True: draft = the target's first `draft_layers` layers
    prompt_len: int
    prompt_dist: str             # "uniform" | "zipf"
    k: int
    max_new: int
    n_requests: int = 1
    prompt_seed: int = 100

    @property
    def draft(self) -> ModelShape:
        return self.target.replace(n_layers=self.draft_layers)


def workload(index: int) -> Workload:
    """The five benchmark configs, numbered 1..5."""
    if index == 1:
        return Workload("cfg1_tiny", family_a(4, 256, 4, 1024, 1024, 128, WDTYPE_F32),
                        1, True, 32, "uniform", 4, 32, 1, 101)
    if index == 2:
        return Workload("cfg2_validate_microbench",
                        family_a(24, 1024, 16, 4096, 32128, 2048 + 16, WDTYPE_BF16),
                        1, True, 2048, "uniform", 8, 0, 1, 102)
    if index == 3:
        return Workload("cfg3_3b", family_b(32, 2560, 32, 32, 80, 6912, 32000, 1024),
                        4, True, 512, "zipf", 4, 256, 1, 103)
    if index == 4:
        return Workload("cfg4_7b", family_b(32, 4096, 32, 8, 128, 11008, 32000, 1536),
                        2, False, 1024, "zipf", 8, 256, 1, 104)
    if index == 5:
        return Workload("cfg5_7b_long", family_b(32, 4096, 32, 8, 128, 11008, 32000, 16384 + 256),
                        2, False, 16384, "zipf", 8, 128, 4, 105)
    raise ValueError("workload index must be 1..5")


# ----------------------------------------------------------------------------
# bf16 bit patterns
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


class WeightSource:
    """Lazily generates the tensors of one model, one tensor at a time.

    backend "numpy": numpy Philox streams on the host (bit-reproducible everywhere).
    backend "torch-cuda": torch's CUDA generator (fast for multi-billion-parameter
    shapes); the host copy handed to the CPU oracle is a device-to-host copy of
    the very tensor given to the GPU path, so both still consume identical bits.

    `layer_alias` maps a layer index to (other_source, other_layer): used for an
    early-exit draft whose layers are the target's own first layers.
    """

    def __init__(self, shape: ModelShape, seed: int, backend: str = "numpy",
                 norm_jitter: float = 0.0, std: float = 0.02,
                 share_globals_with: Optional["WeightSource"] = None,
                 share_layers_with: Optional["WeightSource"] = None):
        self.shape, self.seed, self.backend = shape, int(seed), backend
        self.norm_jitter, self.std = float(norm_jitter), float(std)
        self.share_globals_with = share_globals_with
        self.share_layers_with = share_layers_with
        self._cache: Dict[str, object] = {}

    # -- raw draws ------------------------------------------------------------
    def _key(self, layer: int, name: str):
        if layer < 0:
            return [self.seed, 1_000_000, GLOBAL_TENSORS.index(name)]
        return [self.seed, layer, LAYER_TENSORS.index(name)]

    def _draw_numpy(self, layer: int, name: str) -> np.ndarray:
        shp = self.shape.tensor_shape(name)
        rng = np.random.Generator(np.random.Philox(np.random.SeedSequence(self._key(layer, name))))
        if len(shp) == 1:
            base = 0.0 if name.endswith("_b") else 1.0
            out = np.full(shp, base, dtype=np.float32)
            if self.norm_jitter:
                out += np.float32(self.norm_jitter) * rng.standard_normal(shp, dtype=np.float32)
            return out
        return rng.standard_normal(shp, dtype=np.float32) * np.float32(self.std)

    def _draw_torch(self, layer: int, name: str):
        import torch
        shp = self.shape.tensor_shape(name)
        k = self._key(layer, name)
        g = torch.Generator(device="cuda")
        g.manual_seed((k[0] * 1_000_003 + k[1]) * 64 + k[2])
        if len(shp) == 1:
            base = 0.0 if name.endswith("_b") else 1.0
            out = torch.full(shp, base, dtype=torch.float32, device="cuda")
            if self.norm_jitter:
                out += self.norm_jitter * torch.randn(shp, generator=g, device="cuda")
            return out
        return torch.randn(shp, generator=g, device="cuda", dtype=torch.float32) * self.std

    # -- public ---------------------------------------------------------------
    def _resolve(self, layer: int, name: str):
        if layer < 0 and self.share_globals_with is not None:
            return self.share_globals_with, layer
        if layer >= 0 and self.share_layers_with is not None:
            return self.share_layers_with, layer
        return self, layer

    def is_matrix_bf16(self, name: str) -> bool:
        return self.shape.wdtype == WDTYPE_BF16 and len(self.shape.tensor_shape(name)) == 2

    def torch_tensor(self, layer: int, name: str, device: str = "cpu"):
        """The tensor as a torch tensor (bf16 for matrices of bf16 models, fp32 otherwise)
        on `device`.  Cached, so a shared tensor is one allocation."""
        import torch
        src, layer = self._resolve(layer, name)
        if not src.shape.has_tensor(name):
            return None
        ck = f"{layer}:{name}:{device}"
        if ck in src._cache:
            return src._cache[ck]
        if src.backend == "torch-cuda":
            t = src._draw_torch(layer, name)
            if src.is_matrix_bf16(name):
                t = t.to(torch.bfloat16)
            t = t.to(device)
        else:
            a = src._draw_numpy(layer, name)
            if src.is_matrix_bf16(name):
                bits = f32_to_bf16_bits(a)
                t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(device)
            else:
                t = torch.from_numpy(a).to(device)
        t = t.contiguous()
        src._cache[ck] = t
        return t

    def host_array(self, layer: int, name: str, device_hint: str = "cpu") -> Optional[np.ndarray]:
        """Host copy for the CPU oracle: uint16 bf16 bit patterns for bf16 matrices,
        float32 otherwise.  With the torch-cuda backend this is a device-to-host copy of
        the tensor the GPU path was given."""
        import torch
        src, layer = self._resolve(layer, name)
        if not src.shape.has_tensor(name):
            return None
        if src.backend == "torch-cuda":
            cached = [v for k, v in src._cache.items() if k.startswith(f"{layer}:{name}:")]
            t = (cached[0] if cached else self.torch_tensor(layer, name, "cuda")).cpu()
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).numpy().view(np.uint16)
            return t.numpy()
        a = src._draw_numpy(layer, name)
        return f32_to_bf16_bits(a) if src.is_matrix_bf16(name) else a

    def drop_cache(self):
        self._cache.clear()


def make_sources(wl: Workload, backend: str = "numpy", norm_jitter: float = 0.0,
                 target_seed: int = 0, draft_seed: int = 1):
    """(target_source, draft_source) for a workload.  The draft always shares the
    target's embedding, final norm and LM head; an early-exit draft also shares the
    target's first layers, otherwise its layers come from `draft_seed`."""
    tgt = WeightSource(wl.target, target_seed, backend, norm_jitter)
    if wl.draft_shares_target:
        drf = WeightSource(wl.draft, target_seed, backend, norm_jitter,
                           share_globals_with=tgt, share_layers_with=tgt)
    else:
        drf = WeightSource(wl.draft, draft_seed, backend, norm_jitter, share_globals_with=tgt)
    return tgt, drf


# ----------------------------------------------------------------------------
# token ids
# ----------------------------------------------------------------------------
def uniform_tokens(n: int, vocab: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def zipf_tokens(n: int, vocab: int, seed: int, s: float = 1.1) -> np.ndarray:
    """Bounded Zipf on ranks 1..vocab with P(r) proportional to r^-s, sampled by inverse
    CDF; token id = rank - 1."""
    rng = np.random.default_rng(seed)
    p = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p)
    cdf /= cdf[-1]
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u, side="left"), vocab - 1).astype(np.int32)


def prompt_tokens(wl: Workload, request: int = 0, n: Optional[int] = None) -> np.ndarray:
    n = wl.prompt_len if n is None else n
    seed = wl.prompt_seed + 1000 * request
    if wl.prompt_dist == "uniform":
        return uniform_tokens(n, wl.target.vocab, seed)
    return zipf_tokens(n, wl.target.vocab, seed)


def forced_draft(target_tokens: np.ndarray, a: int, vocab: int, seed: int) -> np.ndarray:
    """A k-token draft whose first `a` tokens equal target_tokens[:a], whose token `a`
    (if a < k) differs from target_tokens[a], and whose later tokens are uniform random.
    `target_tokens` has k+1 entries (the target's greedy continuation)."""
    k = len(target_tokens) - 1
    assert 0 <= a <= k
    rng = np.random.default_rng(seed)
    d = rng.integers(0, vocab, size=k, dtype=np.int64).astype(np.int32)
    d[:a] = np.asarray(target_tokens[:a], dtype=np.int32)
    if a < k:
        d[a] = (int(target_tokens[a]) + 1) % vocab
    return d


def forced_accept_lengths(k: int, n: int, seed: int) -> List[int]:
    """n accept lengths uniform on 0..k."""
    rng = np.random.default_rng(seed)
    return [int(x) for x in rng.integers(0, k + 1, size=n)]
