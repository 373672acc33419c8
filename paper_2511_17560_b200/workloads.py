"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and lays them out; it contains none of the
method's arithmetic (no RoPE, attention, scoring or selection) so that the CUDA
path and the CPU oracle can both be fed from it without sharing any computation.

Values are drawn in fp32 with numpy's default_rng (one sub-stream per tensor) and
rounded once to bfloat16; both sides consume the rounded values.  Arrays returned
here are float32 holding bf16-representable numbers.

Stand-ins: the paper evaluates on LongBench / Needle-in-a-Haystack / Ruler inputs
cut into 512-token chunks with a recompute ratio of 0.15 (Experiments, "Details");
none of those datasets or trained checkpoints is used.  Token ids are uniform over
the vocabulary and weights are N(0, 0.02^2), which keeps the shapes, lengths and
chunk structure of the paper's workloads.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rope_theta: float
    rms_eps: float
    qkv_bias: bool = False
    rope_layout: int = 0


@dataclass(frozen=True)
class RequestShape:
    chunk_lens: Tuple[int, ...]
    n_question: int
    ratio: float
    select_layer: int
    n_system: int = 0  # the first n_system slots (chunk 0) are a system prompt: attendable, never a candidate

    @property
    def n_ctx(self) -> int:
        return int(sum(self.chunk_lens))

    @property
    def n(self) -> int:
        return self.n_ctx + self.n_question

    @property
    def offsets(self) -> Tuple[int, ...]:
        out, o = [], 0
        for t in self.chunk_lens:
            out.append(o)
            o += t
        return tuple(out)


TINY = ModelShape("tiny", 1, 512, 8, 8, 64, 1408, 32000, 1e4, 1e-5)
TINY3 = replace(TINY, name="tiny3", n_layers=3)
TINY_GQA = ModelShape("tiny_gqa", 3, 512, 4, 2, 128, 1408, 32000, 5e5, 1e-5)
TINY_G7 = ModelShape("tiny_g7", 2, 896, 7, 1, 128, 1408, 32000, 1e6, 1e-6, qkv_bias=True)
LLAMA8B = ModelShape("llama3-8b-shaped", 32, 4096, 32, 8, 128, 14336, 128256, 5e5, 1e-5)
QWEN7B = ModelShape("qwen2.5-7b-shaped", 28, 3584, 28, 4, 128, 18944, 152064, 1e6, 1e-6, qkv_bias=True)

MODELS: Dict[str, ModelShape] = {m.name: m for m in (TINY, TINY3, TINY_GQA, TINY_G7, LLAMA8B, QWEN7B)}


def request_for(config: str, seed: int = 0) -> Tuple[ModelShape, RequestShape]:
    """The request shapes of the benchmark configurations (by short name)."""
    if config == "tiny":
        return TINY, RequestShape((128,) * 4, 16, 0.15, 0)
    if config == "tiny3":
        return TINY3, RequestShape((128,) * 4, 16, 0.15, 1)
    if config == "tiny_gqa":
        return TINY_GQA, RequestShape((100, 37, 128, 1, 90), 13, 0.15, 1)
    if config == "tiny_g7":
        return TINY_G7, RequestShape((64, 130, 77), 9, 0.2, 1)
    if config == "llama8b_10x512":
        return LLAMA8B, RequestShape((512,) * 10, 32, 0.15, 1)
    if config == "llama8b_64x512":
        return LLAMA8B, RequestShape((512,) * 64, 32, 0.15, 1)
    if config == "qwen7b_16xU":
        rng = np.random.default_rng([seed, 301])
        lens = tuple(int(x) for x in rng.integers(256, 2049, size=16))
        return QWEN7B, RequestShape(lens, 64, 0.15, 1)
    raise KeyError(config)


def batched_requests(seed: int = 0, n_requests: int = 16, pool: int = 200):
    """Batched-serving workload: pool chunk lengths and, per request, the chunk ids and question length."""
    rng = np.random.default_rng([seed, 501])
    pool_lens = [int(x) for x in rng.integers(256, 1025, size=pool)]
    reqs = []
    for _ in range(n_requests):
        c = int(rng.integers(8, 33))
        ids = [int(x) for x in rng.choice(pool, size=c, replace=False)]
        nq = int(rng.integers(16, 65))
        reqs.append((ids, nq))
    return pool_lens, reqs


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bf16 -> fp32 (format conversion only)."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def _normal(rng, shape, std) -> np.ndarray:
    return bf16_round(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


_W_NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def weight_shapes(m: ModelShape) -> Dict[str, Tuple[int, ...]]:
    qd, kvd = m.n_q_heads * m.head_dim, m.n_kv_heads * m.head_dim
    return {
        "wq": (qd, m.d_model), "wk": (kvd, m.d_model), "wv": (kvd, m.d_model), "wo": (m.d_model, qd),
        "w_gate": (m.d_ff, m.d_model), "w_up": (m.d_ff, m.d_model), "w_down": (m.d_model, m.d_ff),
    }


def make_weights(m: ModelShape, seed: int = 0, std: float = 0.02, norm_jitter: float = 0.0) -> List[Dict[str, np.ndarray]]:
    """Per-layer weight dicts (float32 arrays of bf16-representable values), linear maps stored [out][in]."""
    shapes = weight_shapes(m)
    layers = []
    for l in range(m.n_layers):
        w = {}
        for j, name in enumerate(_W_NAMES):
            rng = np.random.default_rng([seed, 101, l, j])
            w[name] = _normal(rng, shapes[name], std)
        rng = np.random.default_rng([seed, 102, l])
        for name in ("attn_norm", "mlp_norm"):
            g = np.ones(m.d_model, dtype=np.float32)
            if norm_jitter:
                g = g + rng.standard_normal(m.d_model, dtype=np.float32) * np.float32(norm_jitter)
            w[name] = bf16_round(g)
        if m.qkv_bias:
            w["bq"] = _normal(rng, (m.n_q_heads * m.head_dim,), std)
            w["bk"] = _normal(rng, (m.n_kv_heads * m.head_dim,), std)
            w["bv"] = _normal(rng, (m.n_kv_heads * m.head_dim,), std)
        layers.append(w)
    return layers


def make_embeddings(m: ModelShape, n_tokens: int, seed: int = 0, std: float = 0.02, stream: int = 0) -> np.ndarray:
    """Embedding rows of uniformly drawn token ids: [n_tokens][d] float32 (bf16 values).

    Drawing the ids and then the rows of a random table is the same distribution as
    drawing the rows directly except for repeated ids; the table itself is only
    materialised for small vocab*d (it is 1 GiB at Llama width), otherwise rows are
    generated per distinct id from a per-id stream.
    """
    rng = np.random.default_rng([seed, 201, stream])
    ids = rng.integers(0, m.vocab, size=n_tokens)
    out = np.empty((n_tokens, m.d_model), dtype=np.float32)
    cache: Dict[int, np.ndarray] = {}
    for t, tok in enumerate(ids):
        tok = int(tok)
        if tok not in cache:
            cache[tok] = _normal(np.random.default_rng([seed, 202, tok]), (m.d_model,), std)
        out[t] = cache[tok]
    return out


def make_cache_like(m: ModelShape, n_tokens: int, seed: int, stream: int, std: float = 1.0) -> Tuple[np.ndarray, np.ndarray]:
    """Random K and V of cache shape [L][T][Hkv][D] for step-level tests that need no real prefill."""
    rk = np.random.default_rng([seed, 401, stream])
    rv = np.random.default_rng([seed, 402, stream])
    shape = (m.n_layers, n_tokens, m.n_kv_heads, m.head_dim)
    return _normal(rk, shape, std), _normal(rv, shape, std)


# ------------------------------------------------------------------ device-side generators (large configs)


def make_weights_device(m: ModelShape, device, seed: int = 0, std: float = 0.02) -> List[Dict[str, torch.Tensor]]:
    """Same distribution as make_weights, drawn on the device in bf16 (13 GiB at Llama-8B width).

    q/k/v are slices of one [Hq*D + 2*Hkv*D][d] tensor and gate/up of one [2F][d] tensor.
    """
    g = torch.Generator(device=device)
    shapes = weight_shapes(m)
    layers = []
    for l in range(m.n_layers):
        g.manual_seed(seed * 1000003 + l)
        w: Dict[str, torch.Tensor] = {}
        for name in _W_NAMES:
            w[name] = (torch.randn(shapes[name], generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
        w["attn_norm"] = torch.ones(m.d_model, device=device, dtype=torch.bfloat16)
        w["mlp_norm"] = torch.ones(m.d_model, device=device, dtype=torch.bfloat16)
        if m.qkv_bias:
            for name, nrow in (("bq", m.n_q_heads), ("bk", m.n_kv_heads), ("bv", m.n_kv_heads)):
                w[name] = (torch.randn(nrow * m.head_dim, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
        layers.append(w)
    return layers


def make_embeddings_device(m: ModelShape, n_tokens: int, device, seed: int = 0, std: float = 0.02, stream: int = 0) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 7919 + 17 + stream)
    return (torch.randn((n_tokens, m.d_model), generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def make_cache_device(m: ModelShape, n_tokens: int, device, seed: int, stream: int, std: float = 1.0):
    g = torch.Generator(device=device)
    g.manual_seed(seed * 104729 + 31 + stream)
    shape = (m.n_layers, n_tokens, m.n_kv_heads, m.head_dim)
    k = (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    v = (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return k, v


# ------------------------------------------------------------------ planted relevance (32K-context configuration)


def plant_embeddings(x0: torch.Tensor, r: RequestShape, planted_chunks, cosine: float = 0.5, seed: int = 0) -> torch.Tensor:
    """Make the question rows and the rows of `planted_chunks` share a direction (cosine ~ `cosine` with it).

    x0: [n][d] embeddings (any device).  Each affected row keeps its norm: e <- |e| (c u + sqrt(1-c^2) e_perp), u a
    seeded unit vector and e_perp the row's unit component orthogonal to u.  Returns a new bf16 tensor.
    """
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 15485863 + 5)
    u = torch.randn(x0.shape[1], generator=g, dtype=torch.float32)
    u = (u / u.norm()).to(x0.device)
    rows = list(range(r.n_ctx, r.n))
    for c in planted_chunks:
        rows += list(range(r.offsets[c], r.offsets[c] + r.chunk_lens[c]))
    idx = torch.tensor(rows, device=x0.device, dtype=torch.long)
    e = x0[idx].float()
    norm = e.norm(dim=1, keepdim=True)
    perp = e - (e @ u)[:, None] * u[None, :]
    perp = perp / perp.norm(dim=1, keepdim=True)
    out = x0.clone()
    out[idx] = (norm * (cosine * u[None, :] + (1.0 - cosine * cosine) ** 0.5 * perp)).to(x0.dtype)
    return out


def tie_keys_to_queries(w: Dict[str, torch.Tensor], m: ModelShape, rho: float = 0.7, seed: int = 0) -> None:
    """In place: make each KV head's key projection correlate (rho) with the mean of its query heads' projections.

    With independent random Wq and Wk the logit q.k has zero mean whatever the inputs share; tying them lets a
    shared input direction show up as attention, which is what the planted configuration needs.
    """
    G, D = m.n_q_heads // m.n_kv_heads, m.head_dim
    wq, wk = w["wq"], w["wk"]
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 32452843 + 11)
    for h in range(m.n_kv_heads):
        mean_q = wq[h * G * D:(h + 1) * G * D].float().view(G, D, -1).mean(dim=0) * (G ** 0.5)
        noise = wk[h * D:(h + 1) * D].float()
        wk[h * D:(h + 1) * D] = (rho * mean_q + (1.0 - rho * rho) ** 0.5 * noise).to(wk.dtype)
