"""Pins for the oracle's transformer forward pass (paper Section 3.1: tokens -> scores).

The paper prints no numeric example, so the forward pass is pinned to library
implementations that share nothing with the oracle (torch's TransformerEncoderLayer
for the LayerNorm/GELU/learned-position family, HuggingFace's Llama for the
RMSNorm/RoPE/SwiGLU/GQA family) and to closed forms.  Norm gains and biases are
jittered away from 1/0 so that a dropped gain or bias fails.
"""
import numpy as np
import pytest
import torch

from oracle import stairs_oracle as so
from paper_2407_19947_b200 import workloads as wl


def tiny_a(wdtype=wl.WDTYPE_F32, layers=2):
    return wl.family_a(layers, 48, 4, 112, 97, 40, wdtype)


def tiny_b(hq=4, hkv=2, hd=12, wdtype=wl.WDTYPE_F32, layers=2):
    return wl.family_b(layers, 48, hq, hkv, hd, 80, 97, 64, wdtype)


def model_of(shape, seed=3, jitter=0.2, std=0.3):
    src = wl.WeightSource(shape, seed, "numpy", norm_jitter=jitter, std=std)
    return so.OracleModel(shape, src), src


def t64(a):
    return torch.from_numpy(np.asarray(so.widen(a), dtype=np.float64))


# ---------------------------------------------------------------------------------------
# family A against torch.nn.TransformerEncoderLayer (pre-norm, exact GELU, causal mask)
# ---------------------------------------------------------------------------------------
def test_family_a_matches_torch_transformer_encoder_layer():
    shape = tiny_a()
    model, src = model_of(shape)
    seq = wl.uniform_tokens(17, shape.vocab, 5)
    d, f = shape.d_model, shape.d_ff
    x = t64(src.host_array(-1, "tok_emb"))[torch.from_numpy(seq).long()] \
        + t64(src.host_array(-1, "pos_emb"))[: len(seq)]
    mask = torch.nn.Transformer.generate_square_subsequent_mask(len(seq)).double()
    for l in range(shape.n_layers):
        layer = torch.nn.TransformerEncoderLayer(d, shape.n_heads, f, dropout=0.0, activation="gelu",
                                                 layer_norm_eps=shape.norm_eps, batch_first=True,
                                                 norm_first=True, bias=True).double().eval()
        with torch.no_grad():
            layer.self_attn.in_proj_weight.copy_(torch.cat([t64(src.host_array(l, n)) for n in ("wq", "wk", "wv")]))
            layer.self_attn.in_proj_bias.zero_()
            layer.self_attn.out_proj.weight.copy_(t64(src.host_array(l, "wo")))
            layer.self_attn.out_proj.bias.zero_()
            layer.linear1.weight.copy_(t64(src.host_array(l, "w_gate_or_fc1")))
            layer.linear1.bias.zero_()
            layer.linear2.weight.copy_(t64(src.host_array(l, "w_down_or_fc2")))
            layer.linear2.bias.zero_()
            layer.norm1.weight.copy_(t64(src.host_array(l, "norm1_w")))
            layer.norm1.bias.copy_(t64(src.host_array(l, "norm1_b")))
            layer.norm2.weight.copy_(t64(src.host_array(l, "norm2_w")))
            layer.norm2.bias.copy_(t64(src.host_array(l, "norm2_b")))
            x = layer(x[None], src_mask=mask)[0]
    with torch.no_grad():
        h = torch.nn.functional.layer_norm(x, (d,), t64(src.host_array(-1, "final_norm_w")),
                                           t64(src.host_array(-1, "final_norm_b")), shape.norm_eps)
        ref = (h @ t64(src.host_array(-1, "lm_head")).T).numpy()
    got = so.forward_logits(model, seq, all_positions=True)
    assert got.dtype == np.float32 and got.shape == ref.shape
    assert np.abs(got - ref).max() < 2e-4 * max(1.0, np.abs(ref).max())
    # last-position form agrees with the all-positions form
    np.testing.assert_allclose(so.forward_logits(model, seq), got[-1], atol=1e-5)


# ---------------------------------------------------------------------------------------
# family B against HuggingFace Llama (RMSNorm, rotate-half RoPE, GQA, SwiGLU)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("hq,hkv,hd", [(4, 2, 12), (4, 4, 10), (8, 2, 16), (6, 1, 8)])
def test_family_b_matches_huggingface_llama(hq, hkv, hd):
    transformers = pytest.importorskip("transformers")
    shape = tiny_b(hq, hkv, hd)
    model, src = model_of(shape)
    cfg = transformers.LlamaConfig(
        vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ff,
        num_hidden_layers=shape.n_layers, num_attention_heads=hq, num_key_value_heads=hkv,
        head_dim=hd, rms_norm_eps=shape.norm_eps, rope_theta=shape.rope_theta,
        attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
        max_position_embeddings=shape.max_pos, hidden_act="silu", attn_implementation="eager")
    hf = transformers.LlamaForCausalLM(cfg).double().eval()
    names = {"self_attn.q_proj": "wq", "self_attn.k_proj": "wk", "self_attn.v_proj": "wv",
             "self_attn.o_proj": "wo", "mlp.gate_proj": "w_gate_or_fc1", "mlp.up_proj": "w_up",
             "mlp.down_proj": "w_down_or_fc2", "input_layernorm": "norm1_w",
             "post_attention_layernorm": "norm2_w"}
    with torch.no_grad():
        hf.model.embed_tokens.weight.copy_(t64(src.host_array(-1, "tok_emb")))
        hf.model.norm.weight.copy_(t64(src.host_array(-1, "final_norm_w")))
        hf.lm_head.weight.copy_(t64(src.host_array(-1, "lm_head")))
        for l in range(shape.n_layers):
            for hf_name, ours in names.items():
                hf.get_parameter(f"model.layers.{l}.{hf_name}.weight").copy_(t64(src.host_array(l, ours)))
        seq = wl.zipf_tokens(23, shape.vocab, 9)
        ref = hf(torch.from_numpy(seq).long()[None]).logits[0].numpy()
    got = so.forward_logits(model, seq, all_positions=True)
    assert np.abs(got - ref).max() < 2e-4 * max(1.0, np.abs(ref).max())


# ---------------------------------------------------------------------------------------
# closed forms and invariants
# ---------------------------------------------------------------------------------------
class _Override:
    """Weight provider that replaces chosen tensors."""

    def __init__(self, base, repl):
        self.base, self.repl = base, repl

    def host_array(self, layer, name):
        if (layer, name) in self.repl:
            return self.repl[(layer, name)]
        return self.base.host_array(layer, name)


@pytest.mark.parametrize("shape", [tiny_a(layers=1), tiny_b(layers=1)])
def test_zero_query_gives_running_mean_of_values(shape):
    # With Wq = 0 every visible position gets the same weight, so the attention output at
    # position i is the mean of v_0..v_i: a closed form for the mask and the softmax.
    _, src = model_of(shape)
    zero_q = np.zeros(shape.tensor_shape("wq"), np.float32)
    model = so.OracleModel(shape, _Override(src, {(0, "wq"): zero_q}))
    seq = wl.uniform_tokens(9, shape.vocab, 2)
    n = len(seq)
    x0 = so.forward_hidden(model, seq, n_layers=0).astype(np.float64)
    g1 = so.widen(src.host_array(0, "norm1_w")).astype(np.float64)
    if shape.norm == wl.NORM_LAYERNORM:
        b1 = so.widen(src.host_array(0, "norm1_b")).astype(np.float64)
        h = (x0 - x0.mean(-1, keepdims=True)) / np.sqrt(x0.var(-1, keepdims=True) + shape.norm_eps) * g1 + b1
    else:
        h = x0 / np.sqrt((x0 ** 2).mean(-1, keepdims=True) + shape.norm_eps) * g1
    v = h @ so.widen(src.host_array(0, "wv")).astype(np.float64).T           # [n, Hkv*hd]
    v = v.reshape(n, shape.n_kv_heads, shape.head_dim)
    run_mean = np.cumsum(v, axis=0) / np.arange(1, n + 1)[:, None, None]
    group = shape.n_heads // shape.n_kv_heads
    attn = np.repeat(run_mean, group, axis=1).reshape(n, -1)               # query head h <- kv head h//group
    after_attn = x0 + attn @ so.widen(src.host_array(0, "wo")).astype(np.float64).T
    # isolate the attention half of the block by zeroing the MLP's output matrix
    zero_down = np.zeros(shape.tensor_shape("w_down_or_fc2"), np.float32)
    model2 = so.OracleModel(shape, _Override(src, {(0, "wq"): zero_q, (0, "w_down_or_fc2"): zero_down}))
    got = so.forward_hidden(model2, seq, n_layers=1)
    assert np.abs(got - after_attn).max() < 1e-4 * max(1.0, np.abs(after_attn).max())


def test_causality_later_tokens_do_not_change_earlier_logits():
    for shape in (tiny_a(), tiny_b()):
        model, _ = model_of(shape)
        seq = wl.uniform_tokens(12, shape.vocab, 4)
        full = so.forward_logits(model, seq, all_positions=True)
        for cut in (1, 5, 11):
            part = so.forward_logits(model, seq[:cut])
            assert np.abs(part - full[cut - 1]).max() < 1e-4
        seq2 = seq.copy()
        seq2[8:] = (seq2[8:] + 1) % shape.vocab
        full2 = so.forward_logits(model, seq2, all_positions=True)
        assert np.abs(full2[:8] - full[:8]).max() < 1e-4
        assert np.abs(full2[8:] - full[8:]).max() > 1e-3


def test_rope_depends_only_on_relative_position():
    # Rotary scores q_m . k_n depend on m - n only, so a RoPE model (no learned positions)
    # gives the same logits when every position is shifted by a constant.
    shape = tiny_b()
    model, _ = model_of(shape)
    seq = wl.uniform_tokens(10, shape.vocab, 6)
    a = so.logits_from_hidden(model, so.forward_hidden(model, seq))
    b = so.logits_from_hidden(model, so.forward_hidden(model, seq, pos_offset=7))
    assert np.abs(a - b).max() < 2e-3
    # while the learned-position family does change
    shape_a = tiny_a()
    model_a, _ = model_of(shape_a)
    a = so.forward_hidden(model_a, seq)
    b = so.forward_hidden(model_a, seq, pos_offset=7)
    assert np.abs(a - b).max() > 1e-3


def test_rope_is_a_rotation_and_identity_at_position_zero():
    rng = np.random.default_rng(0)
    u = rng.standard_normal((5, 3, 16)).astype(np.float32)
    pos = np.array([0, 1, 2, 50, 1000])
    r = so.rope(u, pos, 1e4)
    np.testing.assert_allclose(r[0], u[0], atol=1e-6)
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(u, axis=-1), rtol=1e-5)
    # pair (i, i + hd/2), angle pos * theta^(-2i/hd): check one element by hand
    i, p = 3, 50
    ang = p * 1e4 ** (-2 * i / 16)
    exp_lo = u[3, 1, i] * np.cos(ang) - u[3, 1, i + 8] * np.sin(ang)
    exp_hi = u[3, 1, i + 8] * np.cos(ang) + u[3, 1, i] * np.sin(ang)
    assert abs(r[3, 1, i] - exp_lo) < 1e-4 and abs(r[3, 1, i + 8] - exp_hi) < 1e-4


def test_norms_and_activations_against_library_routines():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 33)).astype(np.float32) * 3 + 1
    g = rng.standard_normal(33).astype(np.float32)
    b = rng.standard_normal(33).astype(np.float32)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x).double(), (33,), torch.from_numpy(g).double(),
                                         torch.from_numpy(b).double(), 1e-5).numpy()
    np.testing.assert_allclose(so.layer_norm(x, g, b, 1e-5), ref, atol=1e-5)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x).double(), (33,), torch.from_numpy(g).double(), 1e-5).numpy()
    np.testing.assert_allclose(so.rms_norm(x, g, 1e-5), ref, atol=1e-5)
    np.testing.assert_allclose(so.gelu(x), torch.nn.functional.gelu(torch.from_numpy(x).double()).numpy(), atol=1e-6)
    np.testing.assert_allclose(so.silu(x), torch.nn.functional.silu(torch.from_numpy(x).double()).numpy(), atol=1e-6)


def test_zero_layers_is_norm_then_head():
    shape = tiny_b(layers=0)
    model, src = model_of(shape)
    seq = [3, 9]
    e = so.widen(src.host_array(-1, "tok_emb")).astype(np.float64)[9]
    h = e / np.sqrt((e ** 2).mean() + shape.norm_eps) * so.widen(src.host_array(-1, "final_norm_w"))
    ref = so.widen(src.host_array(-1, "lm_head")).astype(np.float64) @ h
    np.testing.assert_allclose(so.forward_logits(model, seq), ref, atol=1e-4)


def test_bf16_models_use_exactly_the_bf16_values():
    shape = tiny_b(wdtype=wl.WDTYPE_BF16)
    src = wl.WeightSource(shape, 3, "numpy", std=0.3)
    bits = src.host_array(0, "wq")
    assert bits.dtype == np.uint16
    wide = so.widen(bits)
    t = src.torch_tensor(0, "wq")
    assert t.dtype == torch.bfloat16
    np.testing.assert_array_equal(wide, t.float().numpy())
    # rounding is to nearest even: compare with torch's own conversion of the fp32 draw
    raw = wl.WeightSource(shape.replace(wdtype=wl.WDTYPE_F32), 3, "numpy", std=0.3).host_array(0, "wq")
    np.testing.assert_array_equal(torch.from_numpy(raw).to(torch.bfloat16).float().numpy(), wide)
