"""Parity at the benchmark configurations' full width and length, in the launch configuration bench.py times.

The oracle cannot run these sizes whole in test time, so each request is checked through (a) exact properties that
hold at any size (the selection is the top-p of the scores the GPU computed; rows outside R keep the re-rotated
chunk values bit for bit; scores vanish outside the candidates and their mass is bounded), (b) position recovery on
sampled rows against the oracle, and (c) one recompute layer at full width and length, teacher-forced, on sampled
rows the oracle computes one by one.  (b) and (c) run on seeded synthetic inputs of the configuration's shapes: no
value the library computed is ever an input of the oracle.  Stacks are truncated to three layers (selection at layer 1) except for one
full-depth run; widths, lengths, chunk structure and ratios are the configurations' own.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import a3_oracle as O
from paper_2511_17560_b200 import workloads as W
from tests.helpers import oracle_model
from tests.test_gpu_steps import KV_MAX, KV_MEAN, check_kv, f64, hidden_rows_scale

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def precompute(eng, m, r, x0):
    """Eq. 1 with the library itself: every chunk alone at local positions (all rows through every layer)."""
    ck, cv = [], []
    for o, t in zip(r.offsets, r.chunk_lens):
        K = torch.zeros((m.n_layers, t, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=DEV)
        V = torch.zeros_like(K)
        X = x0[o:o + t].clone()
        pos = torch.arange(t, dtype=torch.int32, device=DEV)
        for l in range(m.n_layers):
            eng.recompute_layer(l, X, pos, K[l], V[l])
        ck.append(K)
        cv.append(V)
    return ck, cv


class Case:
    def __init__(self, config, layers=3, planted=None, emb_std=0.02, seed=0):
        from paper_2511_17560_b200 import a3
        self.a3 = a3
        m, self.r = W.request_for(config)
        self.m = m = replace(m, n_layers=layers)
        r = self.r
        self.weights = W.make_weights_device(m, DEV, seed)
        self.x0 = W.make_embeddings_device(m, r.n, DEV, seed, std=emb_std)
        if planted:
            W.tie_keys_to_queries(self.weights[r.select_layer], m, 0.7, seed)
            self.x0 = W.plant_embeddings(self.x0, r, planted, 0.5, seed)
        self.eng = a3.A3(m, self.weights, r.n + 8)
        self.ck, self.cv = precompute(self.eng, m, r, self.x0)
        self.tab = a3.chunk_table(self.ck, self.cv, r.offsets)

    def buffers(self):
        m, r = self.m, self.r
        K = torch.zeros((m.n_layers, r.n, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=DEV)
        return K, torch.zeros_like(K)

    def fuse(self, ratio=None):
        r = self.r
        K, V = self.buffers()
        req, out = self.eng.make_request(self.tab, len(self.ck), max(r.chunk_lens), r.n_ctx, r.n_question, self.x0, K, V,
                                         ratio=r.ratio if ratio is None else ratio, select_layer=r.select_layer)
        self.eng.fuse_request(req)
        assert self.eng.device_status() == 0
        return K, V, out

    def oracle_layer(self, l):
        return O.LayerWeights(**{k: v.float().cpu().numpy() for k, v in self.weights[l].items()})


def check_request_properties(c: Case, K, V, out, ratio=None):
    """Everything about a finished request that can be checked exactly at any size."""
    m, r = c.m, c.r
    ratio = r.ratio if ratio is None else ratio
    p = O.recompute_count(ratio, r.n, r.n_ctx)
    rows = out["rows"].cpu().numpy()
    s = out["scores"].cpu().numpy().astype(np.float64)
    assert out["p"] == p and rows.shape[0] == p + r.n_question
    assert rows[p:].tolist() == list(range(r.n_ctx, r.n))
    assert np.all(np.diff(rows) > 0)
    assert rows[:p].tolist() == O.topk_select(s, 0, r.n_ctx, p).tolist()  # bit-exact selection on the GPU's scores
    assert np.isfinite(s).all() and (s >= 0).all() and not s[r.n_ctx:].any()
    total = r.n_question * m.n_q_heads
    assert 0.5 * total < s.sum() <= total * (1 + 1e-5)
    assert torch.isfinite(out["x"].float()).all() and torch.isfinite(K.float()).all() and torch.isfinite(V.float()).all()
    # rows outside R at layers after the selection layer: the re-rotated chunk rows, bit for bit
    Kr, Vr = c.buffers()
    c.eng.rope_rerotate(c.tab, len(c.ck), max(r.chunk_lens), Kr, Vr)
    keep = torch.ones(r.n, dtype=torch.bool, device=DEV)
    keep[out["rows"].long()] = False
    for l in range(r.select_layer + 1, m.n_layers):
        assert torch.equal(K[l][keep], Kr[l][keep]) and torch.equal(V[l][keep], Vr[l][keep])
    return rows, s, Kr, Vr


def check_position_recovery_samples(c: Case, n_samples=64, seed=0):
    """Eq. 2 at the configuration's chunk structure on seeded synthetic chunk caches (nothing the library computed
    goes into the oracle): sampled (layer, chunk, token) rows against the oracle, incl. the last chunk (largest
    offset); V copied bit for bit."""
    m, r = c.m, c.r
    ck, cv = zip(*[W.make_cache_device(m, t, DEV, 7 + seed, i, std=1.2) for i, t in enumerate(r.chunk_lens)])
    tab = c.a3.chunk_table(ck, cv, r.offsets)
    Kr, Vr = c.buffers()
    c.eng.rope_rerotate(tab, len(ck), max(r.chunk_lens), Kr, Vr)
    assert c.eng.device_status() == 0
    rng = np.random.default_rng(seed)
    errs = []
    for i in range(n_samples):
        l = int(rng.integers(0, m.n_layers))
        ch = len(r.chunk_lens) - 1 if i % 4 == 0 else int(rng.integers(0, len(r.chunk_lens)))
        t = int(rng.integers(0, r.chunk_lens[ch]))
        src = ck[ch][l, t].float().cpu().numpy().astype(np.float64)[None]
        want = O.rope_rotate(src, np.array([r.offsets[ch]]), m.rope_theta, m.rope_layout)[0]
        got = f64(Kr[l, r.offsets[ch] + t])
        errs.append(np.abs(got - want))
        assert torch.equal(Vr[l, r.offsets[ch] + t], cv[ch][l, t])
    errs = np.stack(errs)
    assert errs.max() <= KV_MAX and errs.mean() <= KV_MEAN, (errs.max(), errs.mean())


def check_layer_samples(c: Case, layer, rows, n_samples=10, seed=0):
    """One recompute layer at full width/length, teacher-forced on seeded synthetic inputs (hidden rows and a cache
    of unit spread drawn with torch's generator; nothing the library computed goes into the oracle).  The GPU runs
    all carried rows; the oracle projects K and V of all carried rows itself (the cache every row attends over)
    and then recomputes sampled rows one by one."""
    m, r = c.m, c.r
    if rows is None:
        # a seeded selection of the request's size: p random document slots (ascending), then the question slots
        p = O.recompute_count(r.ratio, r.n, r.n_ctx)
        rows = np.concatenate([np.sort(np.random.default_rng(900 + seed).choice(r.n_ctx, size=p, replace=False)), np.arange(r.n_ctx, r.n)])
    M = rows.shape[0]
    g = torch.Generator(device=DEV)
    g.manual_seed(1234 + seed)
    X = torch.randn((M, m.d_model), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    K0 = torch.randn((r.n, m.n_kv_heads, m.head_dim), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    V0 = torch.randn((r.n, m.n_kv_heads, m.head_dim), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    Kc, Vc = K0.clone(), V0.clone()
    pos = torch.from_numpy(rows.astype(np.int32)).to(DEV)
    Xg = X.clone()
    lse = torch.empty((M, m.n_q_heads), dtype=torch.float32, device=DEV)
    c.eng.recompute_layer(layer, Xg, pos, Kc, Vc, lse_out=lse)
    assert c.eng.device_status() == 0
    rng = np.random.default_rng(seed)
    sel = np.unique(np.concatenate([[0, M - 1], rng.choice(M, size=n_samples, replace=False)]))
    w, model = c.oracle_layer(layer), oracle_model(m)
    # the oracle's own cache: the synthetic one with K, V of ALL carried rows projected by the oracle (Eq. 5 writes
    # them before the attention); float32 products of bf16 values in float64 accumulation are exact enough here
    Ko, Vo = f64(K0), f64(V0)
    Xall = f64(X)
    a_all = O.round_bf16(O.rmsnorm(Xall, w.attn_norm, model.rms_eps))
    _, k_all, v_all = O.project_qkv(a_all, w, model, rows, O.round_bf16)
    Ko[rows] = k_all
    Vo[rows] = v_all
    Xo, parts = O.recompute_layer(Xall[sel], rows[sel], w, model, Ko, Vo, rnd=O.round_bf16, return_parts=True)
    check_kv(f64(Kc[pos[sel].long()]), parts["k_exact"], "K rows at full width")
    check_kv(f64(Vc[pos[sel].long()]), parts["v_exact"], "V rows at full width")
    check_kv(f64(Xg[sel]), parts["x_exact"], "hidden rows at full width", scale=hidden_rows_scale(parts["x_exact"]))
    np.testing.assert_allclose(lse[sel].cpu().numpy(), parts["lse"], atol=5e-3)
    # rows outside the carried ones are untouched
    keep = torch.ones(r.n, dtype=torch.bool, device=DEV)
    keep[pos.long()] = False
    assert torch.equal(Kc[keep], K0[keep]) and torch.equal(Vc[keep], V0[keep])


def test_llama8b_10x512_three_layers():
    c = Case("llama8b_10x512")
    K, V, out = c.fuse()
    rows, s, Kr, Vr = check_request_properties(c, K, V, out)
    assert out["p"] == 772
    check_position_recovery_samples(c)
    check_layer_samples(c, 2, None)
    # the full block: all 5152 rows at positions 0..n-1 (launch shape of the leading block), sampled rows
    check_layer_samples(c, 0, np.arange(c.r.n), n_samples=6, seed=1)
    c.eng.close()


def test_llama8b_10x512_extensions_three_layers():
    """The rows built after the hot path, at the benchmark configuration's width and length: scores from the cached
    keys, `ex` eviction inside the request, the value-deviation selector."""
    c = Case("llama8b_10x512")
    m, r = c.m, c.r
    p = O.recompute_count(r.ratio, r.n, r.n_ctx)
    Kr, Vr = c.buffers()
    c.eng.rope_rerotate(c.tab, len(c.ck), max(r.chunk_lens), Kr, Vr)
    # (i) cached-key scores: exact selection on the GPU's own scores, rows outside R untouched at EVERY layer
    K, V = c.buffers()
    req, out = c.eng.make_request(c.tab, len(c.ck), max(r.chunk_lens), r.n_ctx, r.n_question, c.x0, K, V, ratio=r.ratio,
                                  select_layer=r.select_layer, score_source=1)
    c.eng.fuse_request(req)
    assert c.eng.device_status() == 0
    rows = out["rows"].cpu().numpy()
    s = out["scores"].cpu().numpy().astype(np.float64)
    assert rows[:p].tolist() == O.topk_select(s, 0, r.n_ctx, p).tolist() and rows[p:].tolist() == list(range(r.n_ctx, r.n))
    assert 0.5 * r.n_question * m.n_q_heads < s.sum() <= r.n_question * m.n_q_heads * (1 + 1e-5)
    keep = torch.ones(r.n, dtype=torch.bool, device=DEV)
    keep[out["rows"].long()] = False
    assert torch.equal(K[:, keep], Kr[:, keep]) and torch.equal(V[:, keep], Vr[:, keep])
    # (the score kernel itself is checked against the oracle at this size in test_query_scores_parity)
    # (ii) eviction at C = 1024 with pooling: kept sets well-formed, compaction exact, fusion unchanged
    K2, V2 = c.buffers()
    req2, out2 = c.eng.make_request(c.tab, len(c.ck), max(r.chunk_lens), r.n_ctx, r.n_question, c.x0, K2, V2, ratio=r.ratio,
                                    select_layer=r.select_layer, evict_capacity=1024, evict_pool=7)
    c.eng.fuse_request(req2)
    assert c.eng.device_status() == 0
    K0, V0, out0 = c.fuse()
    assert torch.equal(K2, K0) and torch.equal(V2, V0) and torch.equal(out2["x"], out0["x"])
    kept = out2["kept"].cpu().numpy()
    k = 1024 - r.n_question
    assert kept.shape == (m.n_layers, m.n_kv_heads, 1024)
    for l in range(m.n_layers):
        for g in range(m.n_kv_heads):
            kg = kept[l, g]
            assert (np.diff(kg) > 0).all() and kg[k:].tolist() == list(range(r.n_ctx, r.n)) and kg[0] >= 0
            idx = torch.from_numpy(kg.astype(np.int64)).to(DEV)
            assert torch.equal(out2["k_evicted"][l][:, g], K2[l][idx, g]) and torch.equal(out2["v_evicted"][l][:, g], V2[l][idx, g])
    assert len({tuple(kept[1, g].tolist()) for g in range(m.n_kv_heads)}) > 1  # heads keep different tokens
    # (iii) value deviation: scores are the squared distances between cached and true values at the selection layer
    K3, V3 = c.buffers()
    req3, out3 = c.eng.make_request(c.tab, len(c.ck), max(r.chunk_lens), r.n_ctx, r.n_question, c.x0, K3, V3, ratio=r.ratio,
                                    select_layer=r.select_layer, selector=1)
    c.eng.fuse_request(req3)
    assert c.eng.device_status() == 0
    s3 = out3["scores"].cpu().numpy().astype(np.float64)
    rows3 = out3["rows"].cpu().numpy()
    assert rows3[:p].tolist() == O.topk_select(s3, 0, r.n_ctx, p).tolist()
    ls = r.select_layer
    keep3 = torch.ones(r.n, dtype=torch.bool, device=DEV)
    keep3[out3["rows"].long()] = False
    # rows that were NOT recomputed still hold the true values at the selection layer: recompute the distances there
    rng = np.random.default_rng(5)
    cand = np.flatnonzero(keep3[: r.n_ctx].cpu().numpy())
    for i in rng.choice(cand, size=32, replace=False):
        want = float(((f64(V3[ls, i]) - f64(Vr[ls, i])) ** 2).sum())
        assert abs(s3[i] - want) <= 1e-4 * max(want, 1e-6) + 1e-7
    assert s3[: r.chunk_lens[0]].max() <= 1e-3 * max(s3.max(), 1e-9) + 1e-6  # first chunk: cached values are (nearly) the true ones
    c.eng.close()


def test_llama8b_10x512_full_depth_runs_clean():
    c = Case("llama8b_10x512", layers=32)
    K, V, out = c.fuse()
    check_request_properties(c, K, V, out)
    K2, V2, out2 = c.fuse()  # same request again: bit-identical (no atomics, fixed reduction orders)
    assert torch.equal(K, K2) and torch.equal(V, V2) and torch.equal(out["x"], out2["x"]) and torch.equal(out["scores"], out2["scores"])
    c.eng.close()


def test_llama8b_32k_planted_relevance():
    planted = (20, 45)
    c = Case("llama8b_64x512", planted=planted, emb_std=1.0)
    K, V, out = c.fuse()
    rows, s, Kr, Vr = check_request_properties(c, K, V, out)
    assert out["p"] == 4920
    Re = rows[: out["p"]]
    share = np.mean([(r // 512) in planted for r in Re])
    assert share >= 3 * len(planted) / 64, share  # the selection concentrates on the planted chunks
    check_position_recovery_samples(c, seed=2)
    check_layer_samples(c, 2, None, n_samples=6, seed=2)
    # the host-buffer entry on the same request (chunk caches and embeddings in pinned host memory; the embeddings of an
    # input this long travel in row panels and the first block starts on the first): the same bits as the device entry
    m, r = c.m, c.r
    hk = [k.cpu().pin_memory() for k in c.ck]
    hv = [v.cpu().pin_memory() for v in c.cv]
    hx = c.x0.cpu().pin_memory()
    Kh, Vh = c.buffers()
    rq, oh = c.eng.make_request(None, len(hk), 0, r.n_ctx, r.n_question, None, Kh, Vh, ratio=r.ratio, select_layer=r.select_layer)
    M = oh["p"] + r.n_question
    rows_h = torch.empty(M, dtype=torch.int32).pin_memory()
    x_h = torch.empty((M, m.d_model), dtype=torch.bfloat16).pin_memory()
    staging = torch.empty(c.eng.host_staging_bytes(r.n_ctx, r.n), dtype=torch.uint8, device=DEV)
    c.eng.fuse_request_host(rq, hk, hv, hx, rows_h, x_h, staging)
    assert c.eng.device_status() == 0
    assert torch.equal(Kh, K) and torch.equal(Vh, V)
    assert torch.equal(rows_h, out["rows"].cpu()) and torch.equal(x_h, out["x"].cpu())
    c.eng.close()


def test_qwen7b_ragged_ratio_sweep():
    c = Case("qwen7b_16xU")
    assert len(c.r.chunk_lens) == 16 and all(256 <= t <= 2048 for t in c.r.chunk_lens)
    prev = None
    for ratio in (0.05, 0.10, 0.15, 0.30):
        K, V, out = c.fuse(ratio)
        rows, s, Kr, Vr = check_request_properties(c, K, V, out, ratio)
        cur = set(rows[: out["p"]].tolist())
        if prev is not None:
            assert prev <= cur  # nested selections on the same request
        prev = cur
        if ratio == 0.15:
            check_position_recovery_samples(c, seed=3)
            check_layer_samples(c, 2, None, n_samples=6, seed=3)  # G = 7 packing, q/k/v bias
    c.eng.close()


def test_batched_serving_matches_single_requests():
    from paper_2511_17560_b200 import a3
    m = replace(W.LLAMA8B, n_layers=3)
    pool_lens, reqs = W.batched_requests(seed=0)
    assert len(pool_lens) == 200 and len(reqs) == 16
    weights = W.make_weights_device(m, DEV, 0)
    n_max = max(sum(pool_lens[i] for i in ids) + nq for ids, nq in reqs)
    eng = a3.A3(m, weights, n_max + 8)
    used = sorted({i for ids, _ in reqs for i in ids})
    pool = {}
    for i in used:  # only the pool chunks some request uses are prefilled
        t = pool_lens[i]
        r1 = W.RequestShape((t,), 0, 0.15, 1)
        x = W.make_embeddings_device(m, t, DEV, 0, stream=1000 + i)
        ck, cv = precompute(eng, m, r1, x)
        pool[i] = (ck[0], cv[0], x)
    batch, singles, keep = [], [], []
    for j, (ids, nq) in enumerate(reqs):
        lens = tuple(pool_lens[i] for i in ids)
        r = W.RequestShape(lens, nq, 0.15, 1)
        xq = W.make_embeddings_device(m, nq, DEV, 0, stream=5000 + j)
        x0 = torch.cat([pool[i][2] for i in ids] + [xq]).contiguous()
        tab = a3.chunk_table([pool[i][0] for i in ids], [pool[i][1] for i in ids], r.offsets)
        for dest in (batch, singles):
            K = torch.zeros((m.n_layers, r.n, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=DEV)
            V = torch.zeros_like(K)
            req, out = eng.make_request(tab, len(ids), max(lens), r.n_ctx, nq, x0, K, V, ratio=0.15, select_layer=1)
            dest.append((req, out, K, V))
        keep.append((x0, tab))
    eng.fuse_batch([b[0] for b in batch])
    for req, out, K, V in singles:
        eng.fuse_request(req)
    assert eng.device_status() == 0
    for (rb, ob, Kb, Vb), (rs, os_, Ks, Vs) in zip(batch, singles):
        assert torch.equal(Kb, Ks) and torch.equal(Vb, Vs) and torch.equal(ob["x"], os_["x"]) and torch.equal(ob["rows"], os_["rows"])
        s = ob["scores"].cpu().numpy().astype(np.float64)
        p = ob["p"]
        n_ctx = rb.n_ctx
        assert ob["rows"].cpu().numpy()[:p].tolist() == O.topk_select(s, 0, n_ctx, p).tolist()
    eng.close()


def test_first_token_llama_vocabulary():
    """Final norm + 128 256 x 4 096 vocabulary projection + greedy choice at Llama-3-8B size: logits of sampled
    vocabulary rows (and of the chosen one) against the oracle, the choice against the kernel's own logits."""
    from paper_2511_17560_b200 import a3
    from tests.test_gpu_steps import FT_TOL
    m = replace(W.LLAMA8B, n_layers=1)
    eng = a3.A3(m, W.make_weights_device(m, DEV, 0), 64)
    vocab, d = 128256, m.d_model
    g = torch.Generator(device=DEV)
    g.manual_seed(21)
    lm = (torch.randn((vocab, d), device=DEV, generator=g) * 0.02).to(torch.bfloat16)
    x = (torch.randn(d, device=DEV, generator=g) * 3.0).to(torch.bfloat16)
    gain = (1.0 + 0.1 * torch.randn(d, device=DEV, generator=g)).to(torch.bfloat16)
    logits, token = eng.first_token(x, gain, lm)
    assert eng.device_status() == 0
    got = logits.cpu().numpy().astype(np.float64)
    tok = int(token.item())
    assert tok == int(np.flatnonzero(got == got.max())[0])
    rows = np.unique(np.concatenate([np.random.default_rng(3).integers(0, vocab, 4096), [0, 1, vocab - 2, vocab - 1, tok]]))
    want, _ = O.first_token(f64(x), f64(gain), f64(lm[torch.from_numpy(rows).to(DEV)]), m.rms_eps, rnd=O.round_bf16)
    scale = np.sqrt(np.mean(want ** 2))
    assert np.abs(got[rows] - want).max() <= FT_TOL * scale
    # the chosen logit is the largest of the sample in the oracle's arithmetic too (up to the tolerance)
    assert want[np.searchsorted(rows, tok)] >= want.max() - 2 * FT_TOL * scale
    eng.close()


@pytest.mark.parametrize("shape,rows", [(W.LLAMA8B, (804, 4952, 7629, 16640)), (W.QWEN7B, (960, 2754, 9404, 16640))])
def test_persistent_gemms_bit_identical_at_full_width(shape, rows):
    """One layer at the real widths, row counts of the configs and in between (16 640 rows: the token matrix no longer
    stays in L2 and the units of the persistent kernels are walked in groups of feature blocks): the persistent CTA-pair
    GEMMs - gate/up, QKV with its RoPE/scatter epilogue, both residual GEMMs forced onto them, each with the token
    tiling chosen for its shape - against the tile kernels, bit for bit: hidden rows and the K/V cache."""
    from paper_2511_17560_b200 import a3
    m = replace(shape, n_layers=1)
    eng = a3.A3(m, W.make_weights_device(m, DEV, 0), max(rows) + 128)
    try:
        for M in rows:
            kv_len = M + 64
            g = torch.Generator(device=DEV)
            g.manual_seed(M)
            pos = torch.sort(torch.randperm(kv_len, device=DEV, generator=g)[:M]).values.to(torch.int32)
            X0 = torch.randn((M, m.d_model), device=DEV, generator=g).to(torch.bfloat16)
            K = torch.randn((kv_len, m.n_kv_heads, m.head_dim), device=DEV, generator=g).to(torch.bfloat16)
            outs = []
            for sw, rs in ((1, 2), (0, 0)):
                eng.set_option(a3.OPT_SWIGLU_PAIR, sw)
                eng.set_option(a3.OPT_RESIDUAL_T, rs)
                eng.set_option(a3.OPT_QKV_T, sw)
                X, Kc, Vc = X0.clone(), K.clone(), K.clone()
                eng.recompute_layer(0, X, pos, Kc, Vc)
                assert eng.device_status() == 0, M
                outs.append((X, Kc, Vc))
            assert torch.isfinite(outs[0][0].float()).all(), M
            for a, b in zip(outs[0], outs[1]):
                assert torch.equal(a, b), M
    finally:
        eng.set_option(a3.OPT_SWIGLU_PAIR, 1)
        eng.set_option(a3.OPT_RESIDUAL_T, 1)
        eng.set_option(a3.OPT_QKV_T, 1)
        eng.close()
