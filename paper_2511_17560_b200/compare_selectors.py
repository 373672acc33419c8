"""Which rows to recompute: the paper's selector against the ones it is compared with, on synthetic inputs.

SYNTHETIC, SOFT CHECK.  The paper argues (Attention Recovery subsection, discussion of Figure 3; Baselines and Details
paragraphs) that rows chosen by question attention recover the full prefill better than rows chosen by value
deviation (CacheBlend), the first/last tokens of every chunk (LegoLink) or at random.  That claim was made on trained
models and real documents.  Here the same comparison runs on seeded random weights and embeddings, where nothing says
which selector should win: the table shows that every selector runs on the same hot path at equal p and how far each
leaves the fused cache and the question's final hidden state from the full prefill - it is not evidence for or
against the paper's claim.

For one request and one recompute count p (the number of chunk-edge rows, so that all selectors recompute the same
number of rows) it reports, per selector, against the full prefill of the concatenated input on the same kernels:
  hidden_l2   mean over question rows of |x_fused - x_full|_2 of the final hidden state, divided by the mean |x_full|_2
  k_l2, v_l2  mean over layers and context slots of |K_fused - K_full|_2 (|V ...|) per slot, divided by the mean norm
Everything is computed by the library's kernels; torch only subtracts and takes norms of the results.

  python -m paper_2511_17560_b200.compare_selectors [--config tiny3|llama8b_3l] [--edge 10] [--seed 0]
"""
from __future__ import annotations

import argparse
import json
from dataclasses import replace
from typing import Dict, Optional

import numpy as np
import torch

from . import a3
from . import workloads as W

SELECTORS = ("attention", "value_deviation", "chunk_edges", "random")


def _rel_l2(a: torch.Tensor, b: torch.Tensor) -> float:
    """mean row-wise |a - b|_2 over mean |b|_2; rows are the leading dimensions, the last one is the vector."""
    a, b = a.float(), b.float()
    return float((a - b).flatten(0, -2).norm(dim=1).mean() / b.flatten(0, -2).norm(dim=1).mean())


def compare(eng, m, r, x0: torch.Tensor, chunk_k, chunk_v, edge: int, seed: int = 0,
            forced: Optional[Dict[str, np.ndarray]] = None) -> Dict[str, dict]:
    """Runs the request once per selector (and with no recompute at all, and with every row recomputed) and returns the
    table.  `forced`: selector name -> rows to use instead of the library's own choice (tests pin both sides of a
    comparison to one index set this way)."""
    dev = x0.device
    L, n, n_ctx, nq = m.n_layers, r.n, r.n_ctx, r.n_question
    shape = (L, n, m.n_kv_heads, m.head_dim)
    Kf, Vf = torch.zeros(shape, dtype=torch.bfloat16, device=dev), torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    x_full = eng.precompute_chunk(x0.clone(), Kf, Vf)  # the full prefill: Eq. 1 on the whole input
    tab = a3.chunk_table(chunk_k, chunk_v, r.offsets)
    edges = a3.chunk_edge_rows(r.chunk_lens, edge, r.n_system)
    p = int(edges.size)
    rows = {"chunk_edges": edges, "random": a3.random_rows(seed, r.n_system, n_ctx, p)}
    table: Dict[str, dict] = {}

    def run(name, **kw):
        K, V = torch.zeros_like(Kf), torch.zeros_like(Vf)
        req, out = eng.make_request(tab, len(chunk_k), max(r.chunk_lens), n_ctx, nq, x0, K, V, select_layer=r.select_layer,
                                    n_system=r.n_system, **kw)
        eng.fuse_request(req)
        pp = out["p"]
        table[name] = {"p": pp, "hidden_l2": _rel_l2(out["x"][pp:], x_full[n_ctx:]),
                       "k_l2": _rel_l2(K[:, :n_ctx].flatten(2), Kf[:, :n_ctx].flatten(2)),
                       "v_l2": _rel_l2(V[:, :n_ctx].flatten(2), Vf[:, :n_ctx].flatten(2)),
                       "rows": out["rows"][:pp].cpu().numpy()}

    def dev_rows(x):
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(dev)

    run("no_recompute", n_recompute=0)
    for name in SELECTORS:
        if forced is not None and name in forced:
            run(name, forced_re=dev_rows(forced[name]))
        elif name == "attention":
            run(name, n_recompute=p)
        elif name == "value_deviation":
            run(name, n_recompute=p, selector=1)
        else:
            run(name, forced_re=dev_rows(rows[name]))
    run("all_rows", n_recompute=n_ctx - r.n_system)
    assert eng.device_status() == 0
    return table


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="tiny3", choices=["tiny3", "llama8b_3l"])
    ap.add_argument("--edge", type=int, default=0, help="first/last tokens of every chunk (0: as many as give about 15 % of the input)")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    if args.config == "tiny3":
        m, r = W.request_for("tiny3")
        weights = [{k: torch.from_numpy(v).to(torch.bfloat16).to(dev) for k, v in w.items()} for w in W.make_weights(m, args.seed, std=0.05)]
    else:
        m, r = W.request_for("llama8b_10x512")
        m = replace(m, n_layers=3)
        weights = W.make_weights_device(m, dev, seed=args.seed)
    x0 = W.make_embeddings_device(m, r.n, dev, seed=args.seed, std=1.0)
    eng = a3.A3(m, weights, r.n + 8)
    ck, cv = [], []
    for o, t in zip(r.offsets, r.chunk_lens):
        K = torch.zeros((m.n_layers, t, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
        V = torch.zeros_like(K)
        eng.precompute_chunk(x0[o:o + t].clone(), K, V)
        ck.append(K)
        cv.append(V)
    edge = args.edge or max(1, int(round(0.15 * r.n / (2 * len(r.chunk_lens)))))
    table = compare(eng, m, r, x0, ck, cv, edge, args.seed)
    for v in table.values():
        v.pop("rows")
    print(json.dumps({"label": "synthetic, soft check", "config": args.config, "model": m.name, "n_ctx": r.n_ctx, "n_question": r.n_question,
                      "edge_tokens": edge, "table": table}))
    eng.close()


if __name__ == "__main__":
    main()
