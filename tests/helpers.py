"""Glue used by tests only: turn generated inputs into the oracle's types."""
import numpy as np

from oracle import a3_oracle as O
from paper_2511_17560_b200 import workloads as W


def oracle_model(m: W.ModelShape) -> O.Model:
    return O.Model(m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff,
                   rope_theta=m.rope_theta, rms_eps=m.rms_eps, rope_layout=m.rope_layout)


def oracle_weights(layers) -> list:
    return [O.LayerWeights(**{k: np.asarray(v) for k, v in w.items()}) for w in layers]


def make_request(m: W.ModelShape, r: W.RequestShape, seed=0, emb_std=0.02, w_std=0.02, dtype=np.float64, rnd=O.identity):
    """Weights, whole-input embeddings and per-chunk caches prefilled by the oracle (Eq. 1)."""
    model = oracle_model(m)
    weights = oracle_weights(W.make_weights(m, seed, std=w_std))
    x0 = W.make_embeddings(m, r.n, seed, std=emb_std)
    ck, cv = [], []
    for c, (o, t) in enumerate(zip(r.offsets, r.chunk_lens)):
        k, v = O.precompute_chunk(x0[o:o + t], weights, model, dtype=dtype, rnd=rnd)
        ck.append(k)
        cv.append(v)
    return model, weights, x0, ck, cv


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    """mean row-wise |a - b|_2 over mean |b|_2 (the last axis is the vector)."""
    a2, b2 = a.reshape(-1, a.shape[-1]), b.reshape(-1, b.shape[-1])
    return float(np.linalg.norm(a2 - b2, axis=1).mean() / np.linalg.norm(b2, axis=1).mean())


def oracle_selector_table(model, weights, x0, ck, cv, r, edge: int, seed: int = 0, rnd=O.identity):
    """The selector comparison on the oracle: per selector (Eq. 3 attention, value deviation, chunk edges, random) at
    equal p, the distance of the fused cache and of the question's final hidden state from the full prefill."""
    n_ctx, nq = r.n_ctx, r.n_question
    Kf, Vf, Xf = O.full_prefill(x0, weights, model, rnd=rnd)
    edges = O.chunk_edge_rows(r.chunk_lens, edge, r.n_system)
    p = int(edges.size)
    ratio = (p + 0.5) / r.n  # floor(ratio * n) = p
    assert O.recompute_count(ratio, r.n, n_ctx - r.n_system) == p
    table = {}

    def add(name, **kw):
        res = O.fuse_request(ck, cv, x0, nq, weights, model, kw.pop("ratio", ratio), select_layer=r.select_layer, n_system=r.n_system, rnd=rnd, **kw)
        shp = (model.n_layers, n_ctx, -1)
        table[name] = {"p": int(res.Re.size), "rows": res.Re, "hidden_l2": rel_l2(res.X[res.Re.size:], Xf[n_ctx:]),
                       "k_l2": rel_l2(res.K[:, :n_ctx].reshape(shp), Kf[:, :n_ctx].reshape(shp)),
                       "v_l2": rel_l2(res.V[:, :n_ctx].reshape(shp), Vf[:, :n_ctx].reshape(shp))}

    add("no_recompute", ratio=0.0)
    add("attention")
    add("value_deviation", selector="value_deviation")
    add("chunk_edges", forced_Re=edges)
    add("random", forced_Re=O.random_rows(seed, r.n_system, n_ctx, p))
    add("all_rows", ratio=1.0)
    return table
