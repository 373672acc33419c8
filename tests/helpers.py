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
