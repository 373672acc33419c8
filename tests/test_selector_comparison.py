"""The selector comparison (attention, value deviation, chunk edges, random at equal p) - a synthetic, soft check.

On random weights nothing says which selector must win, so these tests pin what IS fixed: the helpers (random rows
against their stated generator, equal counts), the end points (no recompute is the position-recovered concatenation,
all rows reproduce the full prefill), and that the table the library's tool prints is the table the oracle computes
on the same index sets.
"""
import numpy as np
import pytest
import torch

from oracle import a3_oracle as O
from paper_2511_17560_b200 import workloads as W
from tests.helpers import make_request, oracle_selector_table


def test_random_rows_generator():
    """Distinct, in range, ascending, reproducible; the first swap written out by hand from the stated recipe."""
    rows = O.random_rows(5, 10, 110, 30)
    assert rows.size == 30 and len(set(rows.tolist())) == 30 and rows.min() >= 10 and rows.max() < 110
    assert rows.tolist() == sorted(rows.tolist()) and rows.tolist() == O.random_rows(5, 10, 110, 30).tolist()
    assert O.random_rows(6, 10, 110, 30).tolist() != rows.tolist()
    assert O.random_rows(1, 0, 7, 7).tolist() == list(range(7)) and O.random_rows(1, 0, 7, 99).size == 7 and O.random_rows(1, 3, 9, 0).size == 0
    # k = 1: the chosen slot is cand_begin + mix(seed) mod n, with mix multiplied out here step by step
    m64 = (1 << 64) - 1
    z = (42 + 0x9E3779B97F4A7C15) & m64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m64
    z ^= z >> 31
    assert O.random_rows(42, 100, 1100, 1).tolist() == [100 + z % 1000]
    # every candidate is drawn about equally often (k/n = 1/4 over 400 seeds: 100 +- 5 sigma)
    hits = np.zeros(40)
    for seed in range(400):
        hits[O.random_rows(seed * 7919, 0, 40, 10)] += 1
    assert hits.min() > 100 - 5 * np.sqrt(75) and hits.max() < 100 + 5 * np.sqrt(75)


@pytest.fixture(scope="module")
def tiny3_table():
    m, r = W.request_for("tiny3")
    model, weights, x0, ck, cv = make_request(m, r, seed=0, emb_std=1.0, w_std=0.05)
    return m, r, oracle_selector_table(model, weights, x0, ck, cv, r, edge=10)


def test_oracle_selector_table_tiny3(tiny3_table):
    m, r, t = tiny3_table
    p = t["chunk_edges"]["p"]
    assert p == 2 * 10 * len(r.chunk_lens)
    for name in ("attention", "value_deviation", "chunk_edges", "random"):
        assert t[name]["p"] == p, name  # equal p
        assert all(np.isfinite(t[name][k]) for k in ("hidden_l2", "k_l2", "v_l2"))
    # end points: recomputing every row is the full prefill; recomputing none leaves the largest cache error
    assert t["all_rows"]["hidden_l2"] < 1e-9 and t["all_rows"]["k_l2"] < 1e-9 and t["all_rows"]["v_l2"] < 1e-9
    assert t["no_recompute"]["p"] == 0
    for name in ("attention", "value_deviation", "chunk_edges", "random"):
        assert t[name]["v_l2"] < t["no_recompute"]["v_l2"], name
        assert t[name]["k_l2"] < t["no_recompute"]["k_l2"], name
    # value deviation picks, by its definition, the rows whose cached values are farthest off at the selection layer
    assert set(t["value_deviation"]["rows"].tolist()) != set(t["attention"]["rows"].tolist())


@pytest.mark.gpu
def test_library_selector_table_matches_oracle(tiny3_table):
    """The tool's table (library kernels, bf16) against the oracle's (bf16 storage points mirrored) on the oracle's own
    index sets: the losses agree to a few percent; with its own selections the library picks the top-p of its scores."""
    from paper_2511_17560_b200 import a3
    from paper_2511_17560_b200.compare_selectors import compare
    m, r, _ = tiny3_table
    model, weights, x0, ck, cv = make_request(m, r, seed=0, emb_std=1.0, w_std=0.05, rnd=O.round_bf16)
    want = oracle_selector_table(model, weights, x0, ck, cv, r, edge=10, rnd=O.round_bf16)
    dev = torch.device("cuda:0")
    to = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).to(dev)
    layers = W.make_weights(m, 0, std=0.05)
    eng = a3.A3(m, [{k: to(v) for k, v in w.items()} for w in layers], r.n + 8)
    forced = {k: want[k]["rows"] for k in ("attention", "value_deviation", "chunk_edges", "random")}
    got = compare(eng, m, r, to(x0), [to(k) for k in ck], [to(v) for v in cv], edge=10, seed=0, forced=forced)
    assert got["chunk_edges"]["rows"].tolist() == want["chunk_edges"]["rows"].tolist()
    assert got["random"]["rows"].tolist() == want["random"]["rows"].tolist()
    for name in ("no_recompute", "attention", "value_deviation", "chunk_edges", "random"):
        for k in ("hidden_l2", "k_l2", "v_l2"):
            # both sides are distances between two bf16 pipelines (fused vs full prefill); they differ by rounding noise
            assert got[name][k] == pytest.approx(want[name][k], rel=0.1, abs=5e-3), (name, k, got[name][k], want[name][k])
    assert got["all_rows"]["k_l2"] < 1e-2 and got["all_rows"]["v_l2"] < 1e-2
    # the library's own selections (no forcing): same count, and the chunk-edge / random helpers agree with the oracle's
    own = compare(eng, m, r, to(x0), [to(k) for k in ck], [to(v) for v in cv], edge=10, seed=0)
    for name in ("attention", "value_deviation"):
        assert own[name]["p"] == want[name]["p"]
        overlap = len(set(own[name]["rows"].tolist()) & set(want[name]["rows"].tolist())) / want[name]["p"]
        assert overlap > 0.8, (name, overlap)
    eng.close()
