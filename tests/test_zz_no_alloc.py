"""a3_query_scores_static: the workspace-free variant of the score call, for callers that cannot allocate.

Collected last on purpose (file name), so that a run stopping at the first failure has already run every other
test.  The variant must give what a3_query_scores gives on the same inputs - bit for bit, since both run the same
kernels with the same split of the statistics pass - and what the oracle's Eq. 3 gives within the stated 1e-3, on two
calls in a row that share the library's built-in scratch; and it must refuse sizes beyond that scratch.
"""
import numpy as np
import pytest
import torch

from oracle import a3_oracle as O
from paper_2511_17560_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _engine(m):
    from dataclasses import replace
    from paper_2511_17560_b200 import a3
    m1 = replace(m, n_layers=1, d_ff=256, vocab=8)
    dev = torch.device("cuda:0")
    layers = W.make_weights(m1, 0)
    eng = a3.A3(m1, [{k: torch.from_numpy(v).to(torch.bfloat16).to(dev) for k, v in w.items()} for w in layers], 4096)
    return a3, eng, m1, dev


def _inputs(m, n_ctx, nq, seed, dev):
    rng = np.random.default_rng(seed)
    n = n_ctx + nq
    q = torch.from_numpy(rng.standard_normal((nq, m.n_q_heads, m.head_dim), dtype=np.float32) * 1.3).to(torch.bfloat16).to(dev)
    K = torch.from_numpy(rng.standard_normal((n, m.n_kv_heads, m.head_dim), dtype=np.float32) * 1.3).to(torch.bfloat16).to(dev)
    pos = torch.arange(n_ctx, n, dtype=torch.int32, device=dev)
    return q, K, pos


def test_static_variant_matches_workspace_variant_twice_in_a_row():
    a3, eng, m, dev = _engine(W.TINY_GQA)
    model = O.Model(m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.rope_theta, m.rms_eps, m.rope_layout)
    # two different requests back to back: the second is smaller, so stale scratch entries from the first remain
    for n_ctx, nq, n_sys, seed in ((1500, 40, 7, 1), (333, 9, 0, 2)):
        q, K, pos = _inputs(m, n_ctx, nq, seed, dev)
        got = eng.query_scores_static(q, pos, K, n_sys, n_ctx)
        same = eng.query_scores(q, pos, K, n_sys, n_ctx)
        torch.cuda.synchronize()
        assert torch.equal(got, same)  # the same kernels on the same split: bit for bit
        want = O.query_scores(q.float().cpu().numpy().astype(np.float64), pos.cpu().numpy(), K.float().cpu().numpy().astype(np.float64),
                              model, n_sys, n_ctx)
        g = got.cpu().numpy().astype(np.float64)
        assert not g[:n_sys].any() and not g[n_ctx:].any()
        rel = np.abs(g[n_sys:n_ctx] - want[n_sys:n_ctx]) / want[n_sys:n_ctx]
        assert rel.max() <= 1e-3, rel.max()
    assert eng.device_status() == 0
    eng.close()


def test_static_variant_rejects_sizes_beyond_its_scratch():
    a3, eng, m, dev = _engine(W.TINY)
    nq = 65536 // m.n_q_heads + 1
    q, K, pos = _inputs(m, 64, nq, 3, dev)
    scores = torch.full((64 + nq,), -1.0, dtype=torch.float32, device=dev)
    with pytest.raises(a3.A3Error) as e:
        eng.query_scores_static(q, pos, K, 0, 64, scores=scores)
    assert e.value.status == -6 and "limit" in str(e.value)
    torch.cuda.synchronize()
    assert (scores == -1.0).all()  # nothing was launched
    eng.close()
