"""Plain CPU oracle for attention-aware KV-cache fusion (A^3).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what the fusion hot path computes.  It is written from the paper's Method section
and shares nothing with the CUDA library: no kernels, headers, tables, helpers or
constants.  Only the tests, the smoke check and the benchmark's cpu_baseline /
reference arm may import it; the product path never does.

Arithmetic: numpy, float64 by default (``dtype`` may be set to float32).  RoPE
angles are always formed in float64.  A library matmul serves as a step; there is
no blocking, fusion or reordering beyond what the equations state.

Notation follows the paper: chunks i in {S, D_1..D_k} with per-layer caches K_i,
V_i (Eq. 1); the concatenation K_cat, V_cat; position recovery K'_cat = R_{Theta,m}
K_cat (Eq. 2); relevance score s(d_i) and recompute set Re = top_p(s), p = r*n
(Eq. 3); attention of rows [Re, Q] over the fused cache (Eq. 4, Eq. 5).

Readings adopted where the paper is silent (stated once here, used throughout):
  * theta_i = base^(-2i/D), i = 0..D/2-1, D = head dimension, applied per head
    (the paper writes the hidden size h; the printed matrix ends at theta_{h/2-1}).
  * Softmax scale 1/sqrt(D); grouped-query attention: query head h reads KV head
    h // (Hq/Hkv).
  * The decoder block is the standard pre-norm one: RMSNorm, QKV (+optional bias),
    RoPE, causal attention, output projection + residual, RMSNorm, SwiGLU MLP +
    residual.  H(.) in Eq. 5 abbreviates the norm/MLP part.
  * Causal mask: a row at global position m sees cache slots 0..m.
  * s(d_i) sums over all query heads and all question rows; each softmax row is
    taken over every key the question row can see, then restricted to document
    columns (so sum_i s_i <= |Q|*Hq).
  * p = min(#candidates, floor(r*n + 1e-9)), n = |S|+|D|+|Q|.
  * Ties in top_p: higher score first, then lower index; Re is returned ascending.
  * Inside a layer the K/V rows of [Re, Q] are written into the fused cache before
    the attention of that layer is taken (Eq. 5 lists the assignments first).
  * Chunks are stored at chunk-local positions 0..|i|-1 and re-rotated by the
    chunk's offset; by R(a)R(b) = R(a+b) this equals rotating un-encoded keys by
    the global position (Eq. 2).

Pins (tests marked "not gpu"): RoPE composition / R(0)=I / norm / the D=4 matrix
written out by hand; the decoder block (recompute_layer, project_qkv) against a
2-token d=4 block multiplied out with `math` only and against the Llama and
Qwen2 decoder layers of the `transformers` package in float64 (keys, values,
block output, a two-layer stack); layer-0 and chunk-0 exactness of recovered caches against a
full prefill; r=1 == full prefill; r=0 == position-recovered concatenation;
softmax rows sum to one; uniform-key closed form; causality; brute-force top-k;
nested selections; first-token logits against a library matmul and planted rows;
eviction votes summing to Eq. 3's scores, brute-force kept sets, capacity >= n keeps all.  Whole-request agreement of a deep bf16 stack with this oracle
has no pin beyond the oracle itself ("parity unpinned" for that one statement).
"""
from __future__ import annotations

import math
import time
from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------- model


@dataclass
class Model:
    """Shape of the decoder stack (Background section: L layers, hidden size h)."""

    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5
    rope_layout: int = 0  # 0: pairs (i, i+D/2); 1: pairs (2i, 2i+1) as in the printed matrix


@dataclass
class LayerWeights:
    """One decoder block.  Linear maps are stored [out][in] (y = x @ W.T)."""

    attn_norm: np.ndarray
    wq: np.ndarray
    wk: np.ndarray
    wv: np.ndarray
    wo: np.ndarray
    mlp_norm: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    bq: Optional[np.ndarray] = None
    bk: Optional[np.ndarray] = None
    bv: Optional[np.ndarray] = None


def identity(x: np.ndarray) -> np.ndarray:
    return x


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even) and return in x's dtype.

    Used only when a test asks the oracle to mirror the storage points of a bf16
    pipeline (the values a bf16 implementation must write to memory between steps).
    """
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    out = u.astype(np.uint32).view(np.float32)
    return out.astype(x.dtype, copy=False).reshape(x.shape)


# --------------------------------------------------------------------------- RoPE (Eq. 2)


def rope_frequencies(head_dim: int, theta: float) -> np.ndarray:
    """Theta = {theta_i = base^(-2i/D), i = 0..D/2-1} (Position Recovery paragraph)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    return np.power(np.float64(theta), -2.0 * i / np.float64(head_dim))


def rope_cos_sin(pos: np.ndarray, head_dim: int, theta: float):
    """cos(m*theta_i), sin(m*theta_i) for every position m; float64 angles."""
    ang = np.asarray(pos, dtype=np.float64)[:, None] * rope_frequencies(head_dim, theta)[None, :]
    return np.cos(ang), np.sin(ang)


def rope_rotate(x: np.ndarray, pos: np.ndarray, theta: float, layout: int = 0) -> np.ndarray:
    """Apply R_{Theta,m} (the block-diagonal rotation printed before Eq. 2) to x[m, head, :].

    x: [T][H][D]; pos: [T] integer positions m.  Each 2x2 block rotates one pair of
    coordinates by m*theta_i: (a, b) -> (a cos - b sin, a sin + b cos).  layout 1
    pairs coordinates (2i, 2i+1) as printed; layout 0 pairs (i, i+D/2).
    """
    T, H, D = x.shape
    cos, sin = rope_cos_sin(pos, D, theta)
    cos = cos.astype(x.dtype)[:, None, :]
    sin = sin.astype(x.dtype)[:, None, :]
    out = np.empty_like(x)
    if layout == 0:
        a, b = x[..., : D // 2], x[..., D // 2 :]
        out[..., : D // 2] = a * cos - b * sin
        out[..., D // 2 :] = a * sin + b * cos
    else:
        a, b = x[..., 0::2], x[..., 1::2]
        out[..., 0::2] = a * cos - b * sin
        out[..., 1::2] = a * sin + b * cos
    return out


def position_recovery(
    chunk_k: Sequence[np.ndarray],
    chunk_v: Sequence[np.ndarray],
    offsets: Sequence[int],
    n_slots: int,
    model: Model,
    dtype=np.float64,
    rnd: Callable = identity,
    stored_unrotated: bool = False,
):
    """Eq. 2.

    chunk_k[c], chunk_v[c]: [L][T_c][Hkv][D].  Two storage conventions of the
    Position Recovery subsection:
      * stored at chunk-local positions (default): token t of chunk c already
        carries R(t); rotating it by the chunk's offset o_c gives R(o_c + t);
      * stored without positional embedding (stored_unrotated): token t of chunk c
        is rotated by its global position m = o_c + t, which is Eq. 2 as printed.
    V is copied unchanged.  Returns Kf, Vf of shape [L][n_slots][Hkv][D]; slots not
    covered by a chunk (the question rows) are zero.
    """
    L, Hkv, D = model.n_layers, model.n_kv_heads, model.head_dim
    Kf = np.zeros((L, n_slots, Hkv, D), dtype=dtype)
    Vf = np.zeros((L, n_slots, Hkv, D), dtype=dtype)
    for c, (kc, vc) in enumerate(zip(chunk_k, chunk_v)):
        T = kc.shape[1]
        o = int(offsets[c])
        delta = np.full(T, o, dtype=np.int64)
        if stored_unrotated:
            delta = delta + np.arange(T, dtype=np.int64)
        for l in range(L):
            Kf[l, o : o + T] = rnd(rope_rotate(kc[l].astype(dtype), delta, model.rope_theta, model.rope_layout))
            Vf[l, o : o + T] = vc[l].astype(dtype)
    return Kf, Vf


def strip_positions(chunk_k: np.ndarray, model: Model, rnd: Callable = identity) -> np.ndarray:
    """A chunk's keys [L][T][Hkv][D] stored at local positions -> the same keys "without
    positional embedding" (Position Recovery subsection): token t is rotated by -t.
    R(-t) R(t) = I, so this is the key before RoPE."""
    T = chunk_k.shape[1]
    back = -np.arange(T, dtype=np.int64)
    return np.stack([rnd(rope_rotate(chunk_k[l], back, model.rope_theta, model.rope_layout)) for l in range(chunk_k.shape[0])])


# --------------------------------------------------------------------------- block pieces


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain.astype(x.dtype)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def project_qkv(a: np.ndarray, w: LayerWeights, model: Model, pos: np.ndarray, rnd: Callable = identity):
    """Q_l = X_l W^q, K = X_l W^k, V = X_l W^v (Background; Eq. 5), then RoPE on q, k at `pos`."""
    dt = a.dtype
    M = a.shape[0]
    Hq, Hkv, D = model.n_q_heads, model.n_kv_heads, model.head_dim
    q = a @ w.wq.astype(dt).T
    k = a @ w.wk.astype(dt).T
    v = a @ w.wv.astype(dt).T
    if w.bq is not None:
        q = q + w.bq.astype(dt)
    if w.bk is not None:
        k = k + w.bk.astype(dt)
    if w.bv is not None:
        v = v + w.bv.astype(dt)
    q = rope_rotate(q.reshape(M, Hq, D), pos, model.rope_theta, model.rope_layout)
    k = rope_rotate(k.reshape(M, Hkv, D), pos, model.rope_theta, model.rope_layout)
    v = v.reshape(M, Hkv, D)
    return rnd(q), rnd(k), rnd(v)


def attention_probs(q: np.ndarray, pos: np.ndarray, K: np.ndarray, model: Model, head: int) -> np.ndarray:
    """Softmax(q K^T / sqrt(D)) for one query head; row m sees cache slots 0..pos[m]."""
    g = head // (model.n_q_heads // model.n_kv_heads)
    S = (q[:, head, :] @ K[:, g, :].T) / math.sqrt(model.head_dim)
    slots = np.arange(K.shape[0])[None, :]
    S = np.where(slots <= np.asarray(pos)[:, None], S, -np.inf)
    S = S - S.max(axis=1, keepdims=True)
    P = np.exp(S)
    return P / P.sum(axis=1, keepdims=True)


def attention_rows(q: np.ndarray, pos: np.ndarray, K: np.ndarray, V: np.ndarray, model: Model):
    """O = Softmax(Q K'^T / sqrt(D)) V over the fused cache (Eq. 4, Eq. 5).

    q: [M][Hq][D] (already rotated); pos: [M] global positions; K, V: [n][Hkv][D].
    Returns O [M][Hq][D] and the row log-sum-exp [M][Hq] of the scaled logits.
    """
    M = q.shape[0]
    Hq, D = model.n_q_heads, model.head_dim
    gsz = Hq // model.n_kv_heads
    O = np.empty((M, Hq, D), dtype=q.dtype)
    lse = np.empty((M, Hq), dtype=q.dtype)
    slots = np.arange(K.shape[0])[None, :]
    visible = slots <= np.asarray(pos)[:, None]
    for h in range(Hq):
        g = h // gsz
        S = (q[:, h, :] @ K[:, g, :].T) / math.sqrt(D)
        S = np.where(visible, S, -np.inf)
        mx = S.max(axis=1, keepdims=True)
        P = np.exp(S - mx)
        den = P.sum(axis=1, keepdims=True)
        O[:, h, :] = (P / den) @ V[:, g, :]
        lse[:, h] = (mx + np.log(den))[:, 0]
    return O, lse


def recompute_layer(
    X: np.ndarray,
    pos: np.ndarray,
    w: LayerWeights,
    model: Model,
    K: np.ndarray,
    V: np.ndarray,
    rnd: Callable = identity,
    return_parts: bool = False,
):
    """One layer of Eq. 5 for the carried rows (all n rows for a full block).

    X: [M][d] hidden rows at global positions pos (ascending; position = cache slot).
    K, V: this layer's fused cache [n][Hkv][D], updated IN PLACE at rows pos before
    the attention is taken.  Returns the rows' hidden state after the block.
    `rnd` is applied at the points where a bf16 pipeline stores a tensor
    (norm outputs, q/k/v after RoPE, attention output, hidden state after each
    residual, the SwiGLU product); with the default identity nothing is rounded.
    """
    M = X.shape[0]
    a = rnd(rmsnorm(X, w.attn_norm, model.rms_eps))
    q_e, k_e, v_e = project_qkv(a, w, model, pos, identity)  # exact values, before storage rounding
    q, k, v = rnd(q_e), rnd(k_e), rnd(v_e)
    K[pos] = k
    V[pos] = v
    o, lse = attention_rows(q, pos, K, V, model)
    o = rnd(o).reshape(M, model.n_q_heads * model.head_dim)
    X1 = rnd(X + o @ w.wo.astype(X.dtype).T)
    a2 = rnd(rmsnorm(X1, w.mlp_norm, model.rms_eps))
    hmid = rnd(silu(a2 @ w.w_gate.astype(X.dtype).T) * (a2 @ w.w_up.astype(X.dtype).T))
    X2_e = X1 + hmid @ w.w_down.astype(X.dtype).T
    X2 = rnd(X2_e)
    if return_parts:
        # *_exact: the same quantities before the final storage rounding (what a bf16 result is compared with)
        return X2, dict(a=a, q=q, k=k, v=v, o=o, lse=lse, x_attn=X1, a2=a2, h=hmid,
                        q_exact=q_e, k_exact=k_e, v_exact=v_e, x_exact=X2_e)
    return X2


# --------------------------------------------------------------------------- Eq. 1 and the full prefill


def precompute_chunk(x0: np.ndarray, weights: Sequence[LayerWeights], model: Model, dtype=np.float64, rnd: Callable = identity):
    """K_i, V_i = LLM_theta(i) (Eq. 1): prefill one chunk alone at local positions 0..|i|-1.

    x0: [T][d] embedding rows.  Returns K, V of shape [L][T][Hkv][D].
    """
    T = x0.shape[0]
    pos = np.arange(T)
    X = x0.astype(dtype)
    K = np.zeros((model.n_layers, T, model.n_kv_heads, model.head_dim), dtype=dtype)
    V = np.zeros_like(K)
    for l in range(model.n_layers):
        X = recompute_layer(X, pos, weights[l], model, K[l], V[l], rnd)
    return K, V


def full_prefill(x0: np.ndarray, weights: Sequence[LayerWeights], model: Model, dtype=np.float64, rnd: Callable = identity):
    """Full prefill of the concatenated input (the upper-bound setting without reuse).

    Returns K, V [L][n][Hkv][D] and the final hidden state [n][d].
    """
    n = x0.shape[0]
    pos = np.arange(n)
    X = x0.astype(dtype)
    K = np.zeros((model.n_layers, n, model.n_kv_heads, model.head_dim), dtype=dtype)
    V = np.zeros_like(K)
    for l in range(model.n_layers):
        X = recompute_layer(X, pos, weights[l], model, K[l], V[l], rnd)
    return K, V, X


# --------------------------------------------------------------------------- Eq. 3


def query_scores(q: np.ndarray, q_pos: np.ndarray, K: np.ndarray, model: Model, cand_begin: int, cand_end: int) -> np.ndarray:
    """s(d_i) = sum_j Softmax(q_j K_true^T / sqrt(D))|_{d_i}, summed over query heads (Eq. 3).

    q: [nq][Hq][D] rotated question queries at positions q_pos; K: [n][Hkv][D].
    Returns s of length n: the score for slots in [cand_begin, cand_end), zero elsewhere.
    """
    n = K.shape[0]
    s = np.zeros(n, dtype=q.dtype)
    for h in range(model.n_q_heads):
        P = attention_probs(q, q_pos, K, model, h)  # [nq][n], rows sum to 1 over visible keys
        s += P.sum(axis=0)
    s[:cand_begin] = 0
    s[cand_end:] = 0
    return s


def value_deviation_scores(V_true: np.ndarray, V_cached: np.ndarray, cand_begin: int, cand_end: int) -> np.ndarray:
    """The selector the paper compares against (Baselines, CacheBlend): a token's score is the squared
    distance between its concatenated (cached) value and its ground-truth value at the selection layer,
    summed over KV heads and channels.  V_true, V_cached: [n][Hkv][D]; zero outside the candidates."""
    dvi = V_true - V_cached
    s = (dvi * dvi).sum(axis=(1, 2))
    s[:cand_begin] = 0
    s[cand_end:] = 0
    return s


def chunk_edge_rows(chunk_lens: Sequence[int], m: int, n_system: int = 0) -> np.ndarray:
    """The other selector of the comparison (Baselines, LegoLink; Details: the first and last 20 tokens of
    each chunk): slots of the first m and last m tokens of every chunk, ascending, system prompt slots left out."""
    rows = []
    o = 0
    for t in chunk_lens:
        for i in range(t):
            if (i < m or i >= t - m) and o + i >= n_system:
                rows.append(o + i)
        o += t
    return np.array(rows, dtype=np.int64)


def random_rows(seed: int, cand_begin: int, cand_end: int, k: int) -> np.ndarray:
    """The random selection the paper's comparison mentions (Attention Recovery subsection, Figure 3 discussion):
    k distinct candidate slots drawn uniformly, ascending.  The draw is a counter-based partial shuffle, stated here
    so that any implementation can reproduce it: candidates 0..n-1 in a list; for i = 0..k-1 swap entry i with entry
    i + (mix(seed + i) mod (n - i)), mix being the SplitMix64 finaliser on 64-bit unsigned integers; the first k
    entries, sorted, shifted by cand_begin."""
    mask = (1 << 64) - 1
    n = cand_end - cand_begin
    k = max(0, min(int(k), n))
    idx = list(range(n))
    for i in range(k):
        z = (seed + i + 0x9E3779B97F4A7C15) & mask
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        z ^= z >> 31
        j = i + z % (n - i)
        idx[i], idx[j] = idx[j], idx[i]
    return np.array(sorted(cand_begin + t for t in idx[:k]), dtype=np.int64)


def topk_select(s: np.ndarray, cand_begin: int, cand_end: int, k: int) -> np.ndarray:
    """Re = top_p(s): the k candidate slots with the largest score (Eq. 3).

    Ties go to the lower index; the result is sorted ascending.
    """
    cand = np.arange(cand_begin, cand_end)
    k = max(0, min(int(k), cand.size))
    order = sorted(cand.tolist(), key=lambda i: (-float(s[i]), i))
    return np.array(sorted(order[:k]), dtype=np.int64)


def eviction_scores(q: np.ndarray, q_pos: np.ndarray, K: np.ndarray, model: Model, cand_begin: int, cand_end: int) -> np.ndarray:
    """Extension subsection: the attention the question window pays to every cached token, per KV head.

    e[g][i] = sum over question rows j and the query heads h of group g of
    Softmax_row(q_{j,h} K^T / sqrt(D))[i]; zero outside [cand_begin, cand_end).
    Summed over g this is s(d_i) of Eq. 3.  (SnapKV votes with the observation window's
    attention per head; with grouped-query attention the cache has one entry per KV head,
    so the votes of the heads that share it are added.)
    """
    n = K.shape[0]
    G = model.n_q_heads // model.n_kv_heads
    e = np.zeros((model.n_kv_heads, n), dtype=q.dtype)
    for h in range(model.n_q_heads):
        P = attention_probs(q, q_pos, K, model, h)
        e[h // G] += P.sum(axis=0)
    e[:, :cand_begin] = 0
    e[:, cand_end:] = 0
    return e


def pool_scores(e: np.ndarray, cand_begin: int, cand_end: int, width: int) -> np.ndarray:
    """SnapKV's clustering step: every candidate takes the maximum of the scores in the window of `width`
    (odd) candidates centred on it; the window is cut at the candidate range.  width 1 leaves e unchanged."""
    assert width % 2 == 1
    hw = width // 2
    out = np.zeros_like(e)
    for i in range(cand_begin, cand_end):
        lo, hi = max(cand_begin, i - hw), min(cand_end, i + hw + 1)
        out[:, i] = e[:, lo:hi].max(axis=1)
    return out


def evict_layer(q: np.ndarray, q_pos: np.ndarray, K: np.ndarray, V: np.ndarray, model: Model, n_system: int, n_ctx: int,
                capacity: int, pool: int = 1):
    """Extension subsection (`ex`): keep the system prompt S and the question Q whole and, per KV head, the
    top C - |S| - |Q| document tokens by question-window attention (SnapKV's strategy), for one layer.

    q: [|Q|][Hq][D] rotated question queries of this layer at positions q_pos; K, V: [n][Hkv][D].
    Returns (K_c, V_c, kept): K_c, V_c [C'][Hkv][D] with C' = |S| + k + |Q|, k = clamp(C - |S| - |Q|,
    0, number of document tokens); kept [Hkv][C'] the source slot of every kept entry, ascending.
    """
    n = K.shape[0]
    nq = n - n_ctx
    k = max(0, min(n_ctx - n_system, capacity - n_system - nq))
    e = pool_scores(eviction_scores(q, q_pos, K, model, n_system, n_ctx), n_system, n_ctx, pool)
    Hkv = model.n_kv_heads
    C = n_system + k + nq
    kept = np.zeros((Hkv, C), dtype=np.int64)
    Kc = np.zeros((C, Hkv, K.shape[2]), dtype=K.dtype)
    Vc = np.zeros_like(Kc)
    for g in range(Hkv):
        sel = topk_select(e[g], n_system, n_ctx, k)
        kept[g] = np.concatenate([np.arange(n_system), sel, np.arange(n_ctx, n)])
        Kc[:, g] = K[kept[g], g]
        Vc[:, g] = V[kept[g], g]
    return Kc, Vc, kept


def first_token(x_last: np.ndarray, final_norm: np.ndarray, lm_head: np.ndarray, eps: float, rnd: Callable = identity):
    """The first generated token after fusion (the quantity behind the paper's TTFT figures; Inference
    paragraph of the Experiments): final RMSNorm of the last question row's hidden state, the
    vocabulary projection, greedy choice.

    x_last: [d]; final_norm: [d]; lm_head: [vocab][d].  Returns (logits [vocab], token) with ties
    going to the lowest token id.
    """
    a = rnd(rmsnorm(x_last[None, :], final_norm, eps))[0]
    logits = lm_head.astype(a.dtype) @ a
    best = -np.inf
    token = 0
    for i, v in enumerate(logits.tolist()):
        if v > best:
            best, token = v, i
    return logits, token


def recompute_count(ratio: float, n: int, n_candidates: int) -> int:
    """p = r*n with n the whole input length (Eq. 3), floored and clamped to the candidates."""
    return max(0, min(n_candidates, int(math.floor(ratio * n + 1e-9))))


# --------------------------------------------------------------------------- the whole request


@dataclass
class FuseResult:
    K: np.ndarray          # [L][n][Hkv][D] fused keys
    V: np.ndarray          # [L][n][Hkv][D] fused values
    Re: np.ndarray         # [p] selected document slots, ascending
    R: np.ndarray          # [p+|Q|] carried rows: Re then the question rows
    scores: np.ndarray     # [n] s(d_i) on candidates, 0 elsewhere
    X: np.ndarray          # [p+|Q|][d] final hidden rows of R
    trace: dict = field(default_factory=dict)
    evicted: Optional[list] = None  # per layer (K_c, V_c, kept) of the `ex` extension, when a capacity was given


def fuse_request(
    chunk_k: Sequence[np.ndarray],
    chunk_v: Sequence[np.ndarray],
    x0: np.ndarray,
    n_question: int,
    weights: Sequence[LayerWeights],
    model: Model,
    ratio: float,
    select_layer: int = 1,
    n_system: int = 0,
    dtype=np.float64,
    rnd: Callable = identity,
    forced_Re: Optional[np.ndarray] = None,
    keep_trace: bool = False,
    scores_from_cached_keys: bool = False,
    evict_capacity: int = 0,
    evict_pool: int = 1,
    selector: str = "attention",
) -> FuseResult:
    """Attention-aware fusion of independently prefilled chunk caches (Method section).

    chunk_k/chunk_v: per chunk [L][T_c][Hkv][D] at local positions, in input order
    (a system prompt, if any, is chunk 0 and covers slots 0..n_system-1).
    x0: [n][d] embeddings of the whole input X = (S, D, Q); the last n_question rows
    are the question.  `forced_Re` replaces the selection (used by tests that pin
    both sides to one index set).

    scores_from_cached_keys: the cheaper reading of the Attention Recovery subsection.
    The text obtains Q_true, K_true at layer 1 by passing the whole input through
    block 0; here only the question rows are passed through the leading blocks (over
    the position-recovered cache), their queries are scored against the recovered
    cached keys K' of the selection layer, and rows [Re, Q] are then recomputed
    through every layer from the embeddings (Eq. 5 from l = 0), since no true hidden
    state of Re exists at the selection layer.

    selector: "attention" is Eq. 3; "value_deviation" ranks the candidates by the distance between
    cached and true values at the selection layer instead (the comparison method of the Baselines
    paragraph), everything else unchanged.  Index-only selectors (chunk edges, random) go through
    forced_Re.

    evict_capacity > 0 adds the `ex` extension: right after a layer has been recomputed its
    cache is also returned in compact form (evict_layer), the window being that layer's
    question queries.
    """
    L = model.n_layers
    n = x0.shape[0]
    lens = [k.shape[1] for k in chunk_k]
    offsets = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    n_ctx = int(sum(lens))
    assert n_ctx + n_question == n
    cand_begin, cand_end = n_system, n_ctx
    trace = {}
    evicted = [None] * L if evict_capacity > 0 else None

    def layer_step(l, X, rows):
        """One layer for `rows` (whose last n_question entries are the question), then its eviction."""
        if evicted is None:
            return recompute_layer(X, rows, weights[l], model, K[l], V[l], rnd)
        X2, parts = recompute_layer(X, rows, weights[l], model, K[l], V[l], rnd, return_parts=True)
        nq = n_question
        evicted[l] = evict_layer(parts["q"][len(rows) - nq:], rows[len(rows) - nq:], K[l], V[l], model, n_system, n_ctx,
                                 evict_capacity, evict_pool)
        return X2

    stamps = [("start", time.perf_counter())]  # wall-clock per phase, for the CPU baseline report only

    # position recovery (Eq. 2)
    K, V = position_recovery(chunk_k, chunk_v, offsets, n, model, dtype, rnd)
    stamps.append(("position_recovery", time.perf_counter()))

    if scores_from_cached_keys:
        assert selector == "attention"  # no true values exist in this mode
        q_rows = np.arange(n_ctx, n)
        Xq = x0[q_rows].astype(dtype)
        for l in range(select_layer):
            Xq = recompute_layer(Xq, q_rows, weights[l], model, K[l], V[l], rnd)
        w = weights[select_layer]
        a = rnd(rmsnorm(Xq, w.attn_norm, model.rms_eps))
        q_q, k_q, v_q = project_qkv(a, w, model, q_rows, rnd)
        K[select_layer][q_rows] = k_q
        V[select_layer][q_rows] = v_q
        s = query_scores(q_q, q_rows, K[select_layer], model, cand_begin, cand_end)
        p = recompute_count(ratio, n, cand_end - cand_begin)
        Re = topk_select(s, cand_begin, cand_end, p) if forced_Re is None else np.asarray(forced_Re, dtype=np.int64)
        R = np.concatenate([Re, q_rows]).astype(np.int64)
        stamps.append(("selection", time.perf_counter()))
        X = x0[R].astype(dtype)
        for l in range(L):
            if keep_trace:
                trace[f"x_in_{l}"] = X.copy()
            X = layer_step(l, X, R)
            stamps.append((f"recompute_{l}", time.perf_counter()))
        trace["seconds"] = {name: t - stamps[i][1] for i, (name, t) in enumerate(stamps[1:])}
        return FuseResult(K=K, V=V, Re=Re, R=R, scores=s, X=X, trace=trace, evicted=evicted)

    # embedding + leading decoder blocks over the whole input -> true states at the selection layer
    X = x0.astype(dtype)
    all_pos = np.arange(n)
    for l in range(select_layer):
        X = layer_step(l, X, all_pos)
        stamps.append((f"full_block_{l}", time.perf_counter()))

    # true K, V for every row at the selection layer; question queries; scores; Re (Eq. 3)
    w = weights[select_layer]
    a = rnd(rmsnorm(X, w.attn_norm, model.rms_eps))
    q_all, k_all, v_all = project_qkv(a, w, model, all_pos, rnd)
    V_cached = V[select_layer].copy()
    K[select_layer][:] = k_all
    V[select_layer][:] = v_all
    q_rows = np.arange(n_ctx, n)
    if selector == "value_deviation":
        s = value_deviation_scores(V[select_layer], V_cached, cand_begin, cand_end)
    else:
        assert selector == "attention"
        s = query_scores(q_all[q_rows], q_rows, K[select_layer], model, cand_begin, cand_end)
    p = recompute_count(ratio, n, cand_end - cand_begin)
    Re = topk_select(s, cand_begin, cand_end, p) if forced_Re is None else np.asarray(forced_Re, dtype=np.int64)
    R = np.concatenate([Re, q_rows]).astype(np.int64)
    if keep_trace:
        trace["x_select"] = X.copy()
    X = X[R]
    stamps.append(("selection", time.perf_counter()))

    # layers from the selection layer on: only rows [Re, Q] (Eq. 4, Eq. 5)
    for l in range(select_layer, L):
        if keep_trace:
            trace[f"x_in_{l}"] = X.copy()
        X = layer_step(l, X, R)
        stamps.append((f"recompute_{l}", time.perf_counter()))
    trace["seconds"] = {name: t - stamps[i][1] for i, (name, t) in enumerate(stamps[1:])}
    return FuseResult(K=K, V=V, Re=Re, R=R, scores=s, X=X, trace=trace, evicted=evicted)
