"""Pins for the oracle's decoder block (Eq. 5 with H(.) written out; Background: K_l = X_l W^k_l).

`recompute_layer` and `project_qkv` are checked against two things that share nothing with them:
  * a 2-token, d = 4 block multiplied out with `math` only (tests/golden/block_d4.txt, written by
    tests/golden/make_block_d4.py), with biases, non-unit norm gains and two different positions;
  * the decoder layers of the `transformers` package (Llama: no bias; Qwen2: q/k/v bias) on CPU in float64,
    fed the oracle's weights: keys after RoPE, values and the block output on a dense causal prefix.
Every term of the block is visible in one of them: which projection goes through SiLU, both residuals, the sign
and the place of the biases (before the rotation), the norm gains, the order norm -> projection -> RoPE.
"""
import os

import numpy as np
import pytest
import torch

from oracle import a3_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_block_d4():
    vals = {}
    for line in open(os.path.join(GOLDEN, "block_d4.txt")):
        if line.startswith("#"):
            continue
        f = line.split()
        vals.setdefault(f[0], []).append([float(t) for t in f[1:]])
    return {k: np.array(v) for k, v in vals.items()}


def test_block_d4_multiplied_out_by_hand():
    g = _read_block_d4()
    model = O.Model(1, 4, 1, 1, 4, 3, rope_theta=100.0, rms_eps=1e-5, rope_layout=0)
    w = O.LayerWeights(attn_norm=g["g_attn"][0], wq=g["wq"], wk=g["wk"], wv=g["wv"], wo=g["wo"], mlp_norm=g["g_mlp"][0],
                       w_gate=g["wg"], w_up=g["wu"], w_down=g["wd"], bq=g["bq"][0], bk=g["bk"][0], bv=g["bv"][0])
    pos = np.array([3, 7])
    K = np.zeros((8, 1, 4))
    V = np.zeros((8, 1, 4))
    X2, parts = O.recompute_layer(g["x"].copy(), pos, w, model, K, V, return_parts=True)
    np.testing.assert_allclose(K[pos, 0], g["k"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(V[pos, 0], g["v"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(X2, g["x_out"], rtol=0, atol=1e-13)
    # the cache rows of the block are written at the rows' positions and nowhere else
    untouched = np.setdiff1d(np.arange(8), pos)
    assert not K[untouched].any() and not V[untouched].any()
    # project_qkv alone: the same keys and values from the normalised rows
    q, k, v = O.project_qkv(parts["a"], w, model, pos)
    np.testing.assert_allclose(k[:, 0], g["k"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(v[:, 0], g["v"], rtol=0, atol=1e-13)


def _hf_layer(kind, shape, seed):
    """A transformers decoder layer in float64 and the oracle's weights for it (same numbers)."""
    from transformers.models.llama.modeling_llama import LlamaConfig, LlamaDecoderLayer, LlamaRotaryEmbedding
    from transformers.models.qwen2.modeling_qwen2 import Qwen2Config, Qwen2DecoderLayer, Qwen2RotaryEmbedding

    d, Hq, Hkv, D, F, theta, eps = shape
    common = dict(hidden_size=d, intermediate_size=F, num_hidden_layers=1, num_attention_heads=Hq, num_key_value_heads=Hkv,
                  head_dim=D, rms_norm_eps=eps, max_position_embeddings=4096, vocab_size=32, hidden_act="silu",
                  attention_dropout=0.0)
    if kind == "llama":
        cfg = LlamaConfig(**common, attention_bias=False, mlp_bias=False, rope_parameters={"rope_type": "default", "rope_theta": theta})
        layer, rot = LlamaDecoderLayer(cfg, 0), LlamaRotaryEmbedding(cfg)
    else:
        cfg = Qwen2Config(**common, use_sliding_window=False, rope_parameters={"rope_type": "default", "rope_theta": theta})
        layer, rot = Qwen2DecoderLayer(cfg, 0), Qwen2RotaryEmbedding(cfg)
    cfg._attn_implementation = "sdpa"  # the eager path takes its softmax in float32
    # the package's RMSNorm computes in float32 whatever the input type; torch's own module (same definition, gains
    # included) keeps float64, so the comparison can be held to 1e-9 instead of float32 rounding
    layer.input_layernorm = torch.nn.RMSNorm(d, eps=eps)
    layer.post_attention_layernorm = torch.nn.RMSNorm(d, eps=eps)
    layer = layer.double().eval()
    rot = rot.double()
    g = torch.Generator().manual_seed(seed)
    with torch.no_grad():
        for name, prm in layer.named_parameters():
            if name.endswith("layernorm.weight"):
                prm.copy_(1.0 + 0.5 * torch.randn(prm.shape, generator=g, dtype=torch.float64))
            elif name.endswith("bias"):
                prm.copy_(0.5 * torch.randn(prm.shape, generator=g, dtype=torch.float64))
            else:
                prm.copy_(torch.randn(prm.shape, generator=g, dtype=torch.float64) / np.sqrt(prm.shape[1]))
    sd = {k: v.detach().numpy().copy() for k, v in layer.state_dict().items()}
    w = O.LayerWeights(attn_norm=sd["input_layernorm.weight"], wq=sd["self_attn.q_proj.weight"], wk=sd["self_attn.k_proj.weight"],
                       wv=sd["self_attn.v_proj.weight"], wo=sd["self_attn.o_proj.weight"],
                       mlp_norm=sd["post_attention_layernorm.weight"], w_gate=sd["mlp.gate_proj.weight"],
                       w_up=sd["mlp.up_proj.weight"], w_down=sd["mlp.down_proj.weight"],
                       bq=sd.get("self_attn.q_proj.bias"), bk=sd.get("self_attn.k_proj.bias"), bv=sd.get("self_attn.v_proj.bias"))
    model = O.Model(1, d, Hq, Hkv, D, F, rope_theta=theta, rms_eps=eps, rope_layout=0)
    return cfg, layer, rot, w, model


def _hf_forward(cfg, layer, rot, x):
    """Dense causal prefix at positions 0..n-1 through the library layer; returns (K after RoPE, V, output)."""
    from transformers.cache_utils import DynamicCache

    n = x.shape[0]
    hs = torch.from_numpy(x)[None]
    pos = torch.arange(n)[None]
    cache = DynamicCache(config=cfg)
    mask = torch.full((n, n), float("-inf"), dtype=torch.float64).triu(1)[None, None]
    with torch.no_grad():
        cos, sin = rot(hs, pos)
        # the rotary module keeps its inverse frequencies in float32; rebuild cos/sin from float64 angles of the same
        # definition (theta_i = base^(-2i/D)) so that the comparison is not limited by that storage choice
        inv = torch.tensor(O.rope_frequencies(layer.self_attn.head_dim, cfg.rope_parameters["rope_theta"]))
        ang = pos[0][:, None].double() * inv[None, :]
        cos64, sin64 = torch.cat([ang.cos(), ang.cos()], -1)[None], torch.cat([ang.sin(), ang.sin()], -1)[None]
        assert torch.allclose(cos.double(), cos64, atol=1e-3) and torch.allclose(sin.double(), sin64, atol=1e-3)
        out = layer(hs, attention_mask=mask, position_ids=pos, past_key_values=cache, use_cache=True,
                    position_embeddings=(cos64, sin64))
    out = out[0] if isinstance(out, tuple) else out
    if out.dim() == 2:
        out = out[None]
    lyr = cache.layers[0]
    Kh, Vh = lyr.keys[0], lyr.values[0]  # [Hkv][n][D]
    return Kh.permute(1, 0, 2).numpy(), Vh.permute(1, 0, 2).numpy(), out[0].numpy()


HF_CASES = [("llama", (64, 8, 2, 8, 48, 5e5, 1e-5)), ("qwen2", (56, 7, 1, 8, 40, 1e6, 1e-6)), ("qwen2", (64, 4, 4, 16, 24, 1e4, 1e-6))]


@pytest.mark.parametrize("kind,shape", HF_CASES)
def test_block_matches_transformers_decoder_layer(kind, shape):
    cfg, layer, rot, w, model = _hf_layer(kind, shape, seed=11)
    if kind == "qwen2":
        assert w.bq is not None and w.bk is not None and w.bv is not None
    else:
        assert w.bq is None
    n = 13
    x = np.random.default_rng(12).standard_normal((n, shape[0]))
    Kh, Vh, Yh = _hf_forward(cfg, layer, rot, x)
    K = np.zeros((n, model.n_kv_heads, model.head_dim))
    V = np.zeros_like(K)
    Y = O.recompute_layer(x.copy(), np.arange(n), w, model, K, V)
    np.testing.assert_allclose(K, Kh, rtol=0, atol=1e-9)
    np.testing.assert_allclose(V, Vh, rtol=0, atol=1e-9)
    np.testing.assert_allclose(Y, Yh, rtol=0, atol=1e-9)
    # project_qkv on its own (the selection layer calls it outside recompute_layer)
    a = O.rmsnorm(x, w.attn_norm, model.rms_eps)
    q, k, v = O.project_qkv(a, w, model, np.arange(n))
    np.testing.assert_allclose(k, Kh, rtol=0, atol=1e-9)
    np.testing.assert_allclose(v, Vh, rtol=0, atol=1e-9)
    # sparse rows over the dense cache reproduce the dense rows (Eq. 5 for rows [Re, Q] when the cache is true)
    rows = np.array([2, 5, 11, 12])
    K2, V2 = Kh.copy(), Vh.copy()
    Y2 = O.recompute_layer(x[rows].copy(), rows, w, model, K2, V2)
    np.testing.assert_allclose(Y2, Yh[rows], rtol=0, atol=1e-9)
    np.testing.assert_allclose(K2, Kh, rtol=0, atol=1e-9)


def test_full_prefill_matches_transformers_two_layer_stack():
    """Two stacked blocks (the second one's input is the first one's output): the residual stream is carried."""
    cfg0, l0, rot, w0, model = _hf_layer("qwen2", (56, 7, 1, 8, 40, 1e6, 1e-6), seed=21)
    cfg1, l1, _, w1, _ = _hf_layer("qwen2", (56, 7, 1, 8, 40, 1e6, 1e-6), seed=22)
    n = 9
    x = np.random.default_rng(23).standard_normal((n, 56))
    _, _, y0 = _hf_forward(cfg0, l0, rot, x)
    K1h, V1h, y1 = _hf_forward(cfg1, l1, rot, y0)
    m2 = O.Model(2, 56, 7, 1, 8, 40, rope_theta=1e6, rms_eps=1e-6)
    K, V, X = O.full_prefill(x, [w0, w1], m2)
    np.testing.assert_allclose(X, y1, rtol=0, atol=1e-9)
    np.testing.assert_allclose(K[1], K1h, rtol=0, atol=1e-9)
    np.testing.assert_allclose(V[1], V1h, rtol=0, atol=1e-9)
