#!/usr/bin/env python
"""Benchmark of the A^3 fusion hot path: context tokens fused per second on B200.

A step is one whole fusion request (position recovery of all layers, the leading full block, selection, and the
recompute layers) on synthetic inputs of the configured shape.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl a3|reference] [--config NAME] [--ratio R]

Without --config the headline workload is the largest single-GPU request, `llama8b_64x512` (Llama-3-8B-shaped,
64 chunks x 512 tokens = 32 768 context tokens, relevance planted in two chunks), and the other configurations are
measured in the same run and reported under `configs` in the same line: `llama8b_10x512`, the recompute-ratio sweep
of `qwen7b_16xU` (5, 10, 15, 30 %) and the batched-serving workload `llama8b_batch16`.  With --config only that
workload is measured.  N > 1 runs N independent replicas (one process per GPU, launched with
torch.distributed.run); the path has no exchange step, so there is no data-path collective: only the barrier and
the max-over-ranks of the time.  `--impl reference` times the CPU oracle (as it stands, fp32) on the host cores on
a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (read + write) per launch of the dominant kernel classes from the ncu captures summarised under profiles/
# (gemm_kernels_llama8b_2layer.txt: SwiGLU GEMM of a sparse layer, M = 804, and of the full block, M = 5152;
# attention_kernels_*: see that file).  Used for `roofline.traffic` of the workloads they were captured on.
NCU_TRAFFIC = {("llama8b_10x512", "gemm_swiglu"): {"sparse": 243.87e6 + 18.46e6, "full": 389.03e6 + 140.80e6},
               # attention_and_selection_kernels_llama8b_64x512_2layer.txt: sparse rows (4 952) and the full causal block (32 800)
               ("llama8b_64x512", "attention"): {"sparse": 419.97e6 + 35.71e6, "full": 2208.55e6 + 265.24e6}}

METRIC = "context_tokens_fused_per_s"
UNIT = "tokens/s"
HEADLINE = "llama8b_64x512"
PLANTED_CHUNKS = (20, 45)  # the two chunks whose embeddings share a direction with the question's (cosine 0.5)
SWEEP_RATIOS = (0.05, 0.10, 0.15, 0.30)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sustained_mhz": 1300.0}


def load_peaks():
    """Measured peaks of this machine (generated file) and the SM clock the sustained matmul figure was taken at."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            out = {k: float(p[k]) for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained")}
            out["sustained_mhz"] = float(p.get("clocks_under_load", {}).get("sm_mhz_median") or FALLBACK_PEAKS["sustained_mhz"])
            return out, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ algorithmic work of one request


def algorithmic_work(m, r, p, rows):
    """FLOPs / bytes the method must do per request, per kernel class (not what a kernel happens to move)."""
    n, nq, L, ls = r.n, r.n_question, m.n_layers, r.select_layer
    d, D, Hq, Hkv, F = m.d_model, m.head_dim, m.n_q_heads, m.n_kv_heads, m.d_ff
    M = p + nq
    qd, kvd = Hq * D, Hkv * D
    full_rows = n * ls                      # rows through complete blocks before the selection layer
    sparse_rows = M * (L - ls)              # rows through complete blocks from the selection layer on
    w = {}
    w["gemm_qkv"] = 2.0 * d * ((full_rows + sparse_rows) * (qd + 2 * kvd) + n * 2 * kvd + nq * qd)
    w["gemm_residual"] = 2.0 * (full_rows + sparse_rows) * (qd * d + F * d)
    w["gemm_swiglu"] = 2.0 * (full_rows + sparse_rows) * d * 2 * F
    vis_full = n * (n + 1) / 2.0
    vis_q = float(sum(range(r.n_ctx + 1, n + 1)))
    vis_rows = float(np.sum(np.asarray(rows, dtype=np.float64) + 1.0))
    w["attention"] = 4.0 * D * Hq * (ls * vis_full + (L - ls) * vis_rows) + 2.0 * D * Hq * vis_q
    w["scores"] = 2.0 * D * Hq * vis_q
    # position recovery is queued for the layers above the selection layer (the others are recomputed for every row)
    b = {"rerotate": 4.0 * r.n_ctx * kvd * 2 * (L - ls - 1)}
    return w, b


# ------------------------------------------------------------------ clocks


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", str(period_ms),
                                          "-i", str(gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


# ------------------------------------------------------------------ multi-rank plumbing


def dist_setup(n_gpus: int, backend: str = "nccl"):
    """Returns (rank, world, local_rank).  world > 1 only under torch.distributed.run."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return 0, 1, 0
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend)
    return dist.get_rank(), dist.get_world_size(), int(os.environ.get("LOCAL_RANK", "0"))


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank_per_step: float, steps: int, world: int, max_seconds: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling)."""
    return units_per_rank_per_step * steps * world / max_seconds


def workload_config(name, m, r, p, world, ratio=None, extra=None):
    """The `config` object of a JSON line: the same keys in the CUDA arm and in the reference arm."""
    cfg = {"workload": name, "model": m.name, "chunks": len(r.chunk_lens), "n_ctx": r.n_ctx, "n_question": r.n_question,
           "recompute_ratio": r.ratio if ratio is None else ratio, "n_recompute": p, "select_layer": r.select_layer,
           "replicas": world, "layers": m.n_layers,
           "planted_chunks": list(PLANTED_CHUNKS) if name == HEADLINE else None,
           "l2": "inputs larger than L2: every step streams the stack's weights and the fused cache"}
    if extra:
        cfg.update(extra)
    return cfg


# ------------------------------------------------------------------ the CPU oracle arm


def oracle_sample(config: str, seed: int = 0):
    """Inputs of the bounded oracle sample: 3 layers of the stack at full width, random caches of the workload's shape."""
    from dataclasses import replace
    from oracle import a3_oracle as O
    from paper_2511_17560_b200 import workloads as W
    m_full, r = W.request_for(config)
    m = replace(m_full, n_layers=min(3, m_full.n_layers))
    model = O.Model(m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.rope_theta, m.rms_eps, m.rope_layout)
    weights = [O.LayerWeights(**w) for w in W.make_weights(m, seed)]
    x0 = W.make_embeddings_device(m, r.n, "cpu", seed).float().numpy()
    ck, cv = zip(*[W.make_cache_like(replace(m, n_layers=1), t, seed, c, std=1.28) for c, t in enumerate(r.chunk_lens)])
    return dict(O=O, m_full=m_full, m=m, r=r, model=model, weights=weights, x0=x0, ck=ck, cv=cv)


def oracle_strides(n: int, M: int, budget_rows: int):
    """Row strides of the bounded sample: about `budget_rows` rows through the full block and through the recompute layer."""
    return max(1, -(-n // budget_rows)), max(1, -(-M // budget_rows))


def oracle_step(S, stride_full: int = 4, stride_rows: int = 1, stride_q: int = 1):
    """One bounded sample of the request on the oracle (fp32), with the factors that scale it to the whole request.

    Timed pieces, each the oracle's own function: position recovery of one layer (x L); one full block on every
    `stride_full`-th row (x stride_full x select_layer); the selection layer's norm + QKV on every `stride_full`-th row
    (x stride_full), scores (of every `stride_q`-th question row, x stride_q) and top-p at full size; one recompute layer
    on every `stride_rows`-th of the p + |Q| carried rows (x stride_rows x (L - select_layer)).  Returns (measured
    seconds, extrapolated seconds, parts).
    """
    O, m, mf, r, model, weights = S["O"], S["m"], S["m_full"], S["r"], S["model"], S["weights"]
    dt = np.float32
    L, ls = mf.n_layers, min(r.select_layer, m.n_layers - 1)
    n, nq = r.n, r.n_question
    one = O.Model(1, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.rope_theta, m.rms_eps, m.rope_layout)
    meas, t = {}, {}
    c0 = time.perf_counter()
    K, V = O.position_recovery(S["ck"], S["cv"], r.offsets, n, one, dtype=dt)
    meas["position_recovery"] = time.perf_counter() - c0
    t["position_recovery"] = meas["position_recovery"] * L
    K, V = K[0], V[0]
    X = S["x0"].astype(dt)
    sub = np.arange(0, n, stride_full)
    c0 = time.perf_counter()
    if ls > 0:
        O.recompute_layer(X[sub], sub, weights[0], model, K, V)
    meas["full_blocks"] = time.perf_counter() - c0
    t["full_blocks"] = meas["full_blocks"] * stride_full * ls
    c0 = time.perf_counter()
    w = weights[ls]
    a = O.rmsnorm(X[sub], w.attn_norm, model.rms_eps)
    O.project_qkv(a, w, model, sub)
    t_kv = time.perf_counter() - c0
    c0 = time.perf_counter()
    q_rows = np.arange(r.n_ctx, n)
    q_sub = q_rows[::stride_q]
    aq = O.rmsnorm(X[q_sub], w.attn_norm, model.rms_eps)
    q, _, _ = O.project_qkv(aq, w, model, q_sub)
    s = O.query_scores(q, q_sub, K, model, 0, r.n_ctx)
    p = O.recompute_count(r.ratio, n, r.n_ctx)
    Re = O.topk_select(s, 0, r.n_ctx, p)
    t_sel = time.perf_counter() - c0
    meas["selection"] = t_kv + t_sel
    t["selection"] = t_kv * stride_full + t_sel * stride_q
    R = np.concatenate([Re, q_rows])[::stride_rows]
    c0 = time.perf_counter()
    O.recompute_layer(X[R], R, weights[min(ls + 1, m.n_layers - 1)], model, K, V)
    meas["recompute_layers"] = time.perf_counter() - c0
    t["recompute_layers"] = meas["recompute_layers"] * stride_rows * (L - ls)
    return sum(meas.values()), sum(t.values()), t


def oracle_full_request(config: str, seed: int = 0):
    """The oracle's fuse_request on the WHOLE request (every layer, every row; fp32), not extrapolated.  The stack
    cycles through three distinct layers' weights and the chunk caches are random values of the workload's shape:
    the arithmetic, the shapes and the layer count are the request's own, the values do not matter for a timing."""
    from dataclasses import replace
    from oracle import a3_oracle as O
    from paper_2511_17560_b200 import workloads as W
    m, r = W.request_for(config)
    model = O.Model(m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.rope_theta, m.rms_eps, m.rope_layout)
    three = [O.LayerWeights(**w) for w in W.make_weights(replace(m, n_layers=min(3, m.n_layers)), seed)]
    weights = [three[l % len(three)] for l in range(m.n_layers)]
    x0 = W.make_embeddings_device(m, r.n, "cpu", seed).float().numpy()
    ck, cv = zip(*[W.make_cache_like(m, t, seed, c, std=1.28) for c, t in enumerate(r.chunk_lens)])
    t0 = time.perf_counter()
    res = O.fuse_request(ck, cv, x0, r.n_question, weights, model, r.ratio, select_layer=r.select_layer, dtype=np.float32)
    seconds = time.perf_counter() - t0
    return seconds, r, res.trace.get("seconds", {})


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The reference arm: the oracle on the host cores.  A step is one bounded sample of the workload (sized so that
    the run ends within minutes); `ms_per_step` is the measured time of that sample, `value` the metric it
    extrapolates to for the whole request (`extrapolated`: true)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2511_17560_b200 import workloads as W
    config = args.config or HEADLINE
    S = oracle_sample(config)
    m, r = S["m_full"], S["r"]
    p = S["O"].recompute_count(r.ratio, r.n, r.n_ctx)
    # the sample shrinks with the number of steps asked for, so that any --steps/--warmup ends within minutes
    shrink = min(1.0, 25.0 / max(1, args.steps + args.warmup))
    sf, sr = oracle_strides(r.n, p + r.n_question, max(48, int(args.oracle_rows * shrink)))
    sq = max(1, min(r.n_question, int(round(1.0 / shrink))))
    for _ in range(args.warmup):
        oracle_step(S, sf, sr, sq)
    meas, extr, parts = [], [], None
    for _ in range(args.steps):
        a, b, parts = oracle_step(S, sf, sr, sq)
        meas.append(a)
        extr.append(b)
    t_meas, t_extr = float(np.mean(meas)), float(np.mean(extr))
    value = r.n_ctx / t_extr
    sample = (f"per step: position recovery of 1 layer, one full block and the selection-layer QKV on every {sf}-th row, scores "
              f"of every {sq}-th question row + top-p at full size, one recompute layer on every {sr}-th of the p+|Q| rows; scaled to all layers/rows "
              "(extrapolated); oracle in fp32 with random caches of the workload's shape")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t_meas * 1e3, "extrapolated": True, "extrapolated_request_ms": t_extr * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(config, m, r, p, args.gpus),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample,
                             "seconds_by_phase_extrapolated": parts},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------ the CUDA arm


def precompute_chunks(eng, m, lens, offsets, x0, dev):
    """Eq. 1 on the GPU: each chunk alone at local positions 0..T-1 through every layer (same kernels, all rows)."""
    import torch
    ck, cv = [], []
    for o, t in zip(offsets, lens):
        K = torch.zeros((m.n_layers, t, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
        V = torch.zeros_like(K)
        eng.precompute_chunk(x0[o:o + t].clone(), K, V)
        ck.append(K)
        cv.append(V)
    return ck, cv


class Timer:
    """CUDA-event timing of `steps` calls on the launching stream, bracketed by a barrier and a synchronize on both
    sides; the maximum over ranks is returned."""

    def __init__(self, stream, dev):
        import torch
        self.torch, self.stream, self.dev = torch, stream, dev
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def run(self, call, steps, sync_ranks=True):
        torch = self.torch
        if sync_ranks:
            barrier()
        torch.cuda.synchronize()
        self.e0.record(self.stream)
        for _ in range(steps):
            call()
        self.e1.record(self.stream)
        torch.cuda.synchronize()
        if sync_ranks:
            barrier()
        sec = self.e0.elapsed_time(self.e1) / 1e3
        return max_over_ranks(sec, self.dev) if sync_ranks else sec


def kernel_table(prof, steps, flops, bts, peaks, run_mhz):
    """Per kernel class: time per step and achieved rate against the measured peaks.  `frac` is against the sustained
    matmul peak (the kernels run inside a long step), `frac_burst` against the burst figure, and
    `frac_clock_normalised` puts the class time on the SM clock at which the sustained peak was measured
    (time x this pass's median SM MHz / that MHz), so that a pass running at a higher clock is not flattered."""
    kernels = {}
    for name, e in prof.items():
        if not e["launches"]:
            continue
        per_step_ms = e["ms"] / steps
        k = {"launches_per_step": e["launches"] / steps, "ms_per_step": per_step_ms}
        if name in flops:
            ach = flops[name] / (per_step_ms * 1e-3) / 1e12
            k.update(bound="tensor", achieved=ach, unit="TFLOP/s", frac=ach / peaks["bf16_tflops_sustained"],
                     frac_burst=ach / peaks["bf16_tflops"])
            if run_mhz:
                k["frac_clock_normalised"] = k["frac"] * peaks["sustained_mhz"] / run_mhz
        elif name in bts:
            ach = bts[name] / (per_step_ms * 1e-3) / 1e9
            k.update(bound="hbm", achieved=ach, unit="GB/s", frac=ach / peaks["hbm_gbs"])
        kernels[name] = k
    tot_ms = sum(k["ms_per_step"] for k in kernels.values())
    for k in kernels.values():
        k["share"] = k["ms_per_step"] / tot_ms if tot_ms else 0.0
    return kernels


class RequestWorkload:
    """One fusion request of a named configuration on an engine: inputs, chunk caches (Eq. 1 on the same kernels),
    fused-cache buffers and the request descriptor."""

    def __init__(self, a3, eng, name, m, r, dev, seed=0, ratio=None, planted=False, shared=None):
        import torch
        from paper_2511_17560_b200 import workloads as W
        self.name, self.m, self.r, self.eng = name, m, r, eng
        self.ratio = r.ratio if ratio is None else ratio
        if shared is not None:  # the same request at another ratio: inputs and chunk caches are reused
            self.x0, self.ck, self.cv, self.tab = shared.x0, shared.ck, shared.cv, shared.tab
        else:
            self.x0 = W.make_embeddings_device(m, r.n, dev, seed=seed, std=1.0 if planted else 0.02)
            if planted:
                self.x0 = W.plant_embeddings(self.x0, r, PLANTED_CHUNKS, 0.5, seed)
            self.ck, self.cv = precompute_chunks(eng, m, r.chunk_lens, r.offsets, self.x0, dev)
            self.tab = a3.chunk_table(self.ck, self.cv, r.offsets)
        self.K = torch.zeros((m.n_layers, r.n, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
        self.V = torch.zeros_like(self.K)
        self.req, self.out = eng.make_request(self.tab, len(self.ck), max(r.chunk_lens), r.n_ctx, r.n_question, self.x0, self.K, self.V,
                                              ratio=self.ratio, select_layer=r.select_layer)
        self.p = self.out["p"]

    def measure(self, a3, timer, peaks, steps, warmup, local, rank, use_graph=True, want_plain=False):
        """Warm-up, the timed region (K requests through the public call, nothing else on the stream), then the same
        K requests again with the library's per-launch CUDA events on, for the per-class times."""
        import torch
        eng, req, r, m = self.eng, self.req, self.r, self.m
        eng.workspace(eng.request_workspace_bytes(r.n))
        for _ in range(max(warmup, 3)):
            eng.fuse_request(req)
        torch.cuda.synchronize()
        assert eng.device_status() == 0, "device status word set during warm-up"
        a3.launch_count(reset=True)
        eng.fuse_request(req)
        torch.cuda.synchronize()
        launches_per_step = a3.launch_count(reset=True)
        sampler = ClockSampler(local) if rank == 0 else None
        graph = eng.graph_capture(req) if use_graph else None
        torch.cuda.synchronize()
        a3.launch_count(reset=True)
        if graph is not None:
            graph.launch()  # one untimed replay after the capture
            torch.cuda.synchronize()
            a3.launch_count(reset=True)
            seconds = timer.run(graph.launch, steps)
        else:
            seconds = timer.run(lambda: eng.fuse_request(req), steps)
        gpu_launches = a3.launch_count(reset=True)
        clocks = sampler.stop() if sampler else None
        timed_call = ("a3_fuse_request" if graph is None else
                      "a3_graph_launch (the request recorded once by a3_graph_capture; every kernel runs at every replay)")
        other, other_call = None, None
        if graph is not None and want_plain:
            # the same K requests through the other public way of issuing them; the faster of the two is the headline
            # (long kernels: plain launches, whose programmatic dependent launches overlap a kernel's set-up with its
            # predecessor's tail; short kernels: the graph, which has no launch gaps), the other is reported beside it
            sampler = ClockSampler(local) if rank == 0 else None
            other = timer.run(lambda: eng.fuse_request(req), steps)
            other_clocks = sampler.stop() if sampler else None
            other_call = "a3_fuse_request"
            if other < seconds:
                seconds, other = other, seconds
                clocks, other_clocks = other_clocks, clocks
                timed_call, other_call = other_call, timed_call
        a3.launch_count(reset=True)
        assert eng.device_status() == 0, "device status word set during the timed region"
        # second pass: per-launch CUDA events (about 1 ms per request of their own, which is why `value` is not taken here)
        sampler = ClockSampler(local) if rank == 0 else None
        eng.profile_enable(launches_per_step * steps + 16)
        prof_seconds = timer.run(lambda: eng.fuse_request(req), steps, sync_ranks=False)
        prof = eng.profile_read()
        eng.profile_enable(0)
        prof_clocks = sampler.stop() if sampler else None
        a3.launch_count(reset=True)
        if graph is not None:
            graph.close()
        rows = self.out["rows"].cpu().numpy()
        flops, bts = algorithmic_work(m, r, self.p, rows)
        kernels = kernel_table(prof, steps, flops, bts, peaks, (prof_clocks or {}).get("sm_mhz"))
        total = sum(flops.values())
        ms = seconds / steps * 1e3
        tfs = total / (seconds / steps) / 1e12
        res = {"ms_per_step": ms, "tokens_per_s_per_replica": r.n_ctx / (seconds / steps), "seconds": seconds, "gpu_launches": int(gpu_launches),
               "launches_per_step": int(launches_per_step), "clocks": clocks, "profiled_pass": {"request_ms": prof_seconds / steps * 1e3, "clocks": prof_clocks},
               "other_seconds": other, "other_call": other_call, "kernels": kernels, "algorithmic_tflop_per_request": total / 1e12, "request_tflops": tfs,
               "request_frac_of_sustained_peak": tfs / peaks["bf16_tflops_sustained"], "request_frac_of_burst_peak": tfs / peaks["bf16_tflops"],
               "timed_call": timed_call}
        if clocks and clocks.get("sm_mhz"):
            res["request_frac_clock_normalised"] = res["request_frac_of_sustained_peak"] * peaks["sustained_mhz"] / clocks["sm_mhz"]
        if self.name == HEADLINE or (self.r.n_ctx == 32768):
            planted = set(PLANTED_CHUNKS)
            re = rows[: self.p]
            res["planted_share_of_Re"] = float(np.mean([(int(x) // 512) in planted for x in re])) if len(re) else None
        return res

    def roofline(self, res, peaks, peak_src):
        kernels = res["kernels"]
        top = max(kernels, key=lambda nm: kernels[nm]["ms_per_step"])
        tk = kernels[top]
        traffic = None
        t = NCU_TRAFFIC.get((self.name, top))
        if t:
            nf = self.r.select_layer
            # launch-weighted mean over the class's launches: the leading full blocks, then one sparse-row launch per later layer
            traffic = (t["full"] * nf + t["sparse"] * (self.m.n_layers - nf)) / self.m.n_layers
        return {"kernel": top, "bound": tk.get("bound"), "achieved": tk.get("achieved"),
                "peak": peaks["bf16_tflops_sustained"] if tk.get("bound") == "tensor" else peaks["hbm_gbs"],
                "unit": tk.get("unit"), "frac": tk.get("frac"), "frac_burst": tk.get("frac_burst"),
                "frac_clock_normalised": tk.get("frac_clock_normalised"), "traffic": traffic,
                "peak_source": peak_src + " (sustained: the kernel is timed inside a long step); frac_burst is against the burst figure, "
                               "frac_clock_normalised rescales the time to the SM clock the sustained peak was measured at",
                "timing": "CUDA events the library records around every launch, in a second pass of the same K requests",
                "avg_launch_ms": tk["ms_per_step"] / tk["launches_per_step"], "kernels": kernels}


def sub_result(res, world, steps, n_ctx):
    """What a `configs` entry keeps of a measurement."""
    keep = {"ms_per_step": res["ms_per_step"], "value": aggregate_value(n_ctx, steps, world, res["seconds"]), "unit": UNIT, "steps": steps,
            "request_frac_of_sustained_peak": res["request_frac_of_sustained_peak"], "request_frac_of_burst_peak": res["request_frac_of_burst_peak"],
            "request_frac_clock_normalised": res.get("request_frac_clock_normalised"), "algorithmic_tflop_per_request": res["algorithmic_tflop_per_request"],
            "gpu_launches": res["gpu_launches"], "clocks": res["clocks"],
            "kernels": {k: {f: v[f] for f in ("ms_per_step", "achieved", "unit", "frac", "frac_burst", "frac_clock_normalised", "share") if f in v}
                        for k, v in res["kernels"].items()}}
    return keep


def measure_batch(a3, eng, m, dev, timer, peaks, steps, warmup, local, rank, world):
    """Batched serving (16 requests over a pool of 200 precomputed chunks, Llama-shaped): `a3_fuse_batch` timed as one
    step; aggregate context tokens per second and the spread of the single-request latencies."""
    import torch
    from paper_2511_17560_b200 import workloads as W
    pool_lens, reqs = W.batched_requests(seed=0)
    pool = {}
    for i in sorted({i for ids, _ in reqs for i in ids}):  # only the pool chunks some request uses are prefilled
        t = pool_lens[i]
        x = W.make_embeddings_device(m, t, dev, 0, stream=1000 + i)
        K = torch.zeros((m.n_layers, t, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
        V = torch.zeros_like(K)
        eng.precompute_chunk(x.clone(), K, V)
        pool[i] = (K, V, x)
    batch, keep, n_ctx_total, rows_total, flops_total = [], [], 0, 0, 0.0
    for j, (ids, nq) in enumerate(reqs):
        lens = tuple(pool_lens[i] for i in ids)
        r = W.RequestShape(lens, nq, 0.15, 1)
        xq = W.make_embeddings_device(m, nq, dev, 0, stream=5000 + j)
        x0 = torch.cat([pool[i][2] for i in ids] + [xq]).contiguous()
        tab = a3.chunk_table([pool[i][0] for i in ids], [pool[i][1] for i in ids], r.offsets)
        K = torch.zeros((m.n_layers, r.n, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
        V = torch.zeros_like(K)
        req, out = eng.make_request(tab, len(ids), max(lens), r.n_ctx, nq, x0, K, V, ratio=0.15, select_layer=1)
        batch.append((req, out, r))
        keep.append((x0, tab, K, V))
        n_ctx_total += r.n_ctx
        rows_total += out["p"] + nq
    reqs_c = [b[0] for b in batch]
    for _ in range(max(warmup, 3)):
        eng.fuse_batch(reqs_c)
    torch.cuda.synchronize()
    assert eng.device_status() == 0, "device status word set during warm-up"
    for req, out, r in batch:
        flops, _ = algorithmic_work(m, r, out["p"], out["rows"].cpu().numpy())
        flops_total += sum(flops.values())
    a3.launch_count(reset=True)
    sampler = ClockSampler(local) if rank == 0 else None
    seconds = timer.run(lambda: eng.fuse_batch(reqs_c), steps)
    gpu_launches = a3.launch_count(reset=True)
    clocks = sampler.stop() if sampler else None
    assert eng.device_status() == 0, "device status word set during the timed region"
    lat = []
    for req, out, r in batch:  # each request alone, for the latency spread
        eng.fuse_request(req)
        lat.append(timer.run(lambda: eng.fuse_request(req), 1, sync_ranks=False) * 1e3)
    lat_s = sorted(lat)
    tfs = flops_total / (seconds / steps) / 1e12
    res = {"ms_per_step": seconds / steps * 1e3, "value": aggregate_value(n_ctx_total, steps, world, seconds), "unit": UNIT, "steps": steps,
           "config": {"workload": "llama8b_batch16", "model": m.name, "requests": len(batch), "pool_chunks": len(pool_lens),
                      "pool_chunks_used": len(pool), "n_ctx_total": n_ctx_total, "rows_recomputed_total": rows_total, "recompute_ratio": 0.15,
                      "select_layer": 1, "replicas": world, "layers": m.n_layers, "timed_call": "a3_fuse_batch (16 requests, one step)"},
           "request_latency_ms": {"min": lat_s[0], "median": lat_s[len(lat_s) // 2], "max": lat_s[-1]},
           "algorithmic_tflop_per_step": flops_total / 1e12, "request_frac_of_sustained_peak": tfs / peaks["bf16_tflops_sustained"],
           "request_frac_of_burst_peak": tfs / peaks["bf16_tflops"], "gpu_launches": int(gpu_launches), "clocks": clocks, "seconds": seconds}
    if clocks and clocks.get("sm_mhz"):
        res["request_frac_clock_normalised"] = res["request_frac_of_sustained_peak"] * peaks["sustained_mhz"] / clocks["sm_mhz"]
    del keep
    return res


def measure_e2e(eng, wl, timer, steps, world, dev):
    """The same request through the host-buffer entry: pinned chunk caches + embeddings in, rows + hidden rows out,
    every step; the fused cache itself stays on the device (it is what the decode that follows reads)."""
    import torch
    m, r, p = wl.m, wl.r, wl.p
    hk = [k.cpu().pin_memory() for k in wl.ck]
    hv = [v.cpu().pin_memory() for v in wl.cv]
    hx = wl.x0.cpu().pin_memory()
    rows_h = torch.empty(p + r.n_question, dtype=torch.int32).pin_memory()
    x_h = torch.empty((p + r.n_question, m.d_model), dtype=torch.bfloat16).pin_memory()
    staging = torch.empty(eng.host_staging_bytes(r.n_ctx, r.n), dtype=torch.uint8, device=dev)
    req_h, out_h = eng.make_request(None, len(hk), 0, r.n_ctx, r.n_question, None, wl.K, wl.V, ratio=wl.ratio, select_layer=r.select_layer)
    for _ in range(2):
        eng.fuse_request_host(req_h, hk, hv, hx, rows_h, x_h, staging)
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    sec_dev = timer.run(lambda: eng.fuse_request_host(req_h, hk, hv, hx, rows_h, x_h, staging), steps, sync_ranks=False)
    wall = time.perf_counter() - t0
    sec_e = max_over_ranks(max(sec_dev, wall), dev)
    copied_layers = m.n_layers - r.select_layer - 1  # caches of layers <= select_layer are recomputed, not copied
    h2d = sum(k.numel() * 2 for k in hk) * 2 * copied_layers // m.n_layers + hx.numel() * 2
    d2h = rows_h.numel() * 4 + x_h.numel() * 2
    assert torch.equal(rows_h, wl.out["rows"].cpu()), "host entry selected different rows"
    return {"value": aggregate_value(r.n_ctx, steps, world, sec_e), "unit": UNIT, "ms_per_step": sec_e / steps * 1e3,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "copied": "in: chunk caches of the layers above the selection layer + embeddings, from pinned host memory; out: R and the final "
                      "hidden rows; the fused cache stays on the device"}


def measure_context(eng, wl, timer, peaks, req_ms):
    """Context for the paper's TTFT comparison, on the same kernels: the full prefill of the concatenated input, the
    cheaper reading of the selection, the `ex` eviction, and the first token."""
    import torch
    m, r, p = wl.m, wl.r, wl.p
    dev = wl.K.device
    Kp, Vp = torch.zeros_like(wl.K), torch.zeros_like(wl.V)
    eng.precompute_chunk(wl.x0.clone(), Kp, Vp)
    torch.cuda.synchronize()
    xs = [wl.x0.clone() for _ in range(2)]
    it = iter(xs)
    full_prefill_ms = timer.run(lambda: eng.precompute_chunk(next(it), Kp, Vp), len(xs), sync_ranks=False) / len(xs) * 1e3
    del Kp, Vp, xs

    def variant(**kw):
        req_v, out_v = eng.make_request(wl.tab, len(wl.ck), max(r.chunk_lens), r.n_ctx, r.n_question, wl.x0, wl.K, wl.V, ratio=wl.ratio,
                                        select_layer=r.select_layer, **kw)
        for _ in range(2):
            eng.fuse_request(req_v)
        return timer.run(lambda: eng.fuse_request(req_v), 3, sync_ranks=False) / 3 * 1e3, out_v

    cached_ms, out_c = variant(score_source=1)
    overlap = len(set(out_c["rows"][:p].tolist()) & set(wl.out["rows"][:p].tolist())) / max(p, 1)
    evict_ms, out_e = variant(evict_capacity=1024, evict_pool=7)
    del out_e
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    lm_head = (torch.randn((m.vocab, m.d_model), device=dev, generator=g) * 0.02).to(torch.bfloat16)
    fnorm = torch.ones(m.d_model, dtype=torch.bfloat16, device=dev)
    x_last = wl.out["x"][-1]
    for _ in range(3):
        eng.first_token(x_last, fnorm, lm_head, want_logits=False)
    first_token_ms = timer.run(lambda: eng.first_token(x_last, fnorm, lm_head, want_logits=False), 10, sync_ranks=False) / 10 * 1e3
    first_token_gbs = m.vocab * m.d_model * 2 / (first_token_ms * 1e-3) / 1e9
    del lm_head
    # the standalone HBM-streaming steps of Eq. 4 / Eq. 5 (row gather, K/V scatter) on a synthetic case far beyond the L2:
    # 65 536 rows into / out of 262 144 slots; bytes = rows read + rows written
    n_big, m_big = 262144, 65536
    g.manual_seed(9)
    slots = torch.sort(torch.randperm(n_big, device=dev, generator=g)[:m_big]).values.to(torch.int32)
    kr = torch.randn((m_big, m.n_kv_heads, m.head_dim), device=dev, generator=g).to(torch.bfloat16)
    Kc = torch.zeros((n_big, m.n_kv_heads, m.head_dim), dtype=torch.bfloat16, device=dev)
    Vc = torch.zeros_like(Kc)
    vr = torch.randn((m_big, m.n_kv_heads, m.head_dim), device=dev, generator=g).to(torch.bfloat16)
    eng.scatter_kv(kr, vr, slots, Kc, Vc)
    scatter_s = timer.run(lambda: eng.scatter_kv(kr, vr, slots, Kc, Vc), 10, sync_ranks=False) / 10
    scatter_gbs = 4.0 * m_big * m.n_kv_heads * m.head_dim * 2 / scatter_s / 1e9
    del Vc, kr, vr
    src = Kc.view(-1)[: (n_big // 4) * m.d_model].view(n_big // 4, m.d_model)  # any rows will do: [65 536][d]
    rows = torch.sort(torch.randperm(n_big // 4, device=dev, generator=g)[: m_big // 4]).values.to(torch.int32)
    dst = torch.empty((m_big // 4, m.d_model), dtype=torch.bfloat16, device=dev)
    eng.gather_rows(src, rows, dst)
    gather_s = timer.run(lambda: eng.gather_rows(src, rows, dst), 10, sync_ranks=False) / 10
    gather_gbs = 2.0 * (m_big // 4) * m.d_model * 2 / gather_s / 1e9
    del Kc, src, dst
    return {"hbm_steps": {"scatter_kv": {"rows": m_big, "achieved_gbs": scatter_gbs, "frac_of_hbm_peak": scatter_gbs / peaks["hbm_gbs"]},
                          "gather_rows": {"rows": m_big // 4, "achieved_gbs": gather_gbs, "frac_of_hbm_peak": gather_gbs / peaks["hbm_gbs"]}},
            "full_prefill_ms": full_prefill_ms, "speedup_vs_full_prefill": full_prefill_ms / req_ms,
            "scores_from_cached_keys": {"request_ms": cached_ms, "tokens_per_s": r.n_ctx / (cached_ms * 1e-3),
                                        "selection_overlap_with_true_keys": overlap},
            "ex_eviction": {"capacity": 1024, "pool": 7, "request_ms": evict_ms, "overhead_ms": evict_ms - req_ms},
            "first_token": {"ms": first_token_ms, "achieved_gbs": first_token_gbs, "frac_of_hbm_peak": first_token_gbs / peaks["hbm_gbs"],
                            "ttft_fused_ms": req_ms + first_token_ms, "ttft_full_prefill_ms": full_prefill_ms + first_token_ms,
                            "ttft_ratio": (full_prefill_ms + first_token_ms) / (req_ms + first_token_ms)}}


def run_a3(args):
    import torch
    from dataclasses import replace
    from paper_2511_17560_b200 import a3
    from paper_2511_17560_b200 import workloads as W

    rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks, peak_src = load_peaks()
    suite = args.config is None            # default run: the headline workload plus the other configurations
    main_name = args.config or HEADLINE
    stream = torch.cuda.Stream()           # not the default stream: a graph cannot be recorded there
    torch.cuda.set_stream(stream)
    timer = Timer(stream, dev)
    steps, warmup = args.steps, max(args.warmup, 3)
    sub_steps = max(1, min(steps, 5))

    if main_name == "llama8b_batch16":
        m = W.LLAMA8B if not args.layers else replace(W.LLAMA8B, n_layers=args.layers)
        pool_lens, reqs = W.batched_requests(seed=0)
        n_max = max(sum(pool_lens[i] for i in ids) + nq for ids, nq in reqs)
        eng = a3.A3(m, W.make_weights_device(m, dev, seed=0), n_max + 8)
        res = measure_batch(a3, eng, m, dev, timer, peaks, steps, warmup, local, rank, world)
        if rank == 0:
            line = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
                    "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                    "data": "synthetic", **{k: v for k, v in res.items() if k not in ("value", "unit", "steps", "ms_per_step", "seconds")}}
            print(json.dumps(line), flush=True)
        eng.close()
        return

    m, r = W.request_for(main_name)
    if args.layers:
        m = replace(m, n_layers=args.layers)  # profiling captures only: a truncated stack is not a bench result
    planted = main_name == HEADLINE
    n_max = r.n
    if suite:
        pool_lens, breqs = W.batched_requests(seed=0)
        n_max = max(n_max, max(sum(pool_lens[i] for i in ids) + nq for ids, nq in breqs))
    weights = W.make_weights_device(m, dev, seed=0)
    if planted:
        W.tie_keys_to_queries(weights[r.select_layer], m, 0.7, 0)  # lets a shared input direction show up as attention
    eng = a3.A3(m, weights, n_max + 8)
    wl = RequestWorkload(a3, eng, main_name, m, r, dev, ratio=args.ratio, planted=planted)
    res = wl.measure(a3, timer, peaks, steps, warmup, local, rank, use_graph=not args.no_graph, want_plain=True)
    value = aggregate_value(r.n_ctx, steps, world, res["seconds"])
    roofline = wl.roofline(res, peaks, peak_src)
    e2e = None if args.no_e2e else measure_e2e(eng, wl, timer, steps, world, dev)
    context = {} if args.no_context else measure_context(eng, wl, timer, peaks, res["ms_per_step"])

    configs = {}
    if suite:
        # ---- the other configurations, same library, same run (sub-results; their own lines with --config NAME)
        del wl.ck, wl.cv, wl.K, wl.V
        torch.cuda.empty_cache()
        m2, r2 = W.request_for("llama8b_10x512")
        w2 = RequestWorkload(a3, eng, "llama8b_10x512", m2, r2, dev)
        res2 = w2.measure(a3, timer, peaks, sub_steps, 3, local, rank)
        configs["llama8b_10x512"] = {**sub_result(res2, world, sub_steps, r2.n_ctx), "config": workload_config("llama8b_10x512", m2, r2, w2.p, world)}
        del w2
        torch.cuda.empty_cache()
        b = measure_batch(a3, eng, m, dev, timer, peaks, max(1, min(steps, 3)), 3, local, rank, world)
        b.pop("seconds", None)
        configs["llama8b_batch16"] = b
        eng.close()
        del eng, weights
        torch.cuda.empty_cache()
        m3, r3 = W.request_for("qwen7b_16xU")
        eng3 = a3.A3(m3, W.make_weights_device(m3, dev, seed=0), r3.n + 8)
        sweep, base = {}, None
        for ratio in SWEEP_RATIOS:
            w3 = RequestWorkload(a3, eng3, "qwen7b_16xU", m3, r3, dev, ratio=ratio, shared=base)
            base = base or w3
            res3 = w3.measure(a3, timer, peaks, sub_steps, 3, local, rank)
            sweep[f"{int(round(ratio * 100))}%"] = {**sub_result(res3, world, sub_steps, r3.n_ctx), "n_recompute": w3.p}
        configs["qwen7b_16xU"] = {"config": workload_config("qwen7b_16xU", m3, r3, None, world, ratio=list(SWEEP_RATIOS)), "ratio_sweep": sweep}
        eng3.close()
        del eng3, base, w3
        torch.cuda.empty_cache()
    else:
        eng.close()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        S = oracle_sample(main_name)
        sf, sr = oracle_strides(r.n, wl.p + r.n_question, 4 * args.oracle_rows)
        t_meas, t_extr, parts = oracle_step(S, sf, sr)
        cpu = {"value": r.n_ctx / t_extr, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "seconds": t_extr, "measured_seconds": t_meas,
               "extrapolated": True,
               "sample": f"one bounded oracle step (fp32): 1 layer of position recovery, a full block and the selection QKV on every {sf}-th row, "
                         f"scores + top-p at full size, one recompute layer on every {sr}-th carried row; extrapolated to the whole request",
               "seconds_by_phase": parts}
        del S
        if suite:
            # the whole Llama-shaped 10 x 512 request on the oracle, every layer and row, not extrapolated
            sec, rr, phases = oracle_full_request("llama8b_10x512")
            by = {"position_recovery": phases.get("position_recovery", 0.0), "selection": phases.get("selection", 0.0),
                  "full_blocks": sum(v for k, v in phases.items() if k.startswith("full_block")),
                  "recompute_layers": sum(v for k, v in phases.items() if k.startswith("recompute_"))}
            configs["llama8b_10x512"]["cpu_baseline"] = {"value": rr.n_ctx / sec, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                                         "seconds": sec, "extrapolated": False, "seconds_by_phase": by,
                                                         "sample": "the oracle's fuse_request on the whole request (32 layers, all rows, fp32)"}
    if rank == 0:
        cfg = workload_config(main_name, m, r, wl.p, world, ratio=wl.ratio)  # the same object the reference arm prints
        notes = {"truncated_for_profiling": bool(args.layers), "planted_share_of_Re": res.get("planted_share_of_Re"),
                 "embeddings": "unit-RMS rows; question and planted chunks share a direction (cosine 0.5); key projection of the "
                               "selection layer tied to the query projections (rho 0.7)" if planted else "N(0, 0.02^2) rows"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
                "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic", "config": cfg, "workload_notes": notes,
                "request_ms": res["ms_per_step"], "profiled_pass": res["profiled_pass"], "timed_call": res["timed_call"],
                "other_call": None if res["other_seconds"] is None else
                              {"call": res["other_call"], "ms_per_step": res["other_seconds"] / steps * 1e3,
                               "value": aggregate_value(r.n_ctx, steps, world, res["other_seconds"])},
                **context,
                "algorithmic_tflop_per_request": res["algorithmic_tflop_per_request"], "request_tflops": res["request_tflops"],
                "request_frac_of_sustained_peak": res["request_frac_of_sustained_peak"],
                "request_frac_of_burst_peak": res["request_frac_of_burst_peak"],
                "request_frac_clock_normalised": res.get("request_frac_clock_normalised"),
                "gpu_launches": res["gpu_launches"], "clocks": res["clocks"], "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu,
                "configs": configs or None}
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="a3", choices=["a3", "reference"])
    ap.add_argument("--config", default=None, help="one workload only: llama8b_10x512, llama8b_64x512, qwen7b_16xU, llama8b_batch16, tiny, ...")
    ap.add_argument("--ratio", type=float, default=None, help="recompute ratio of the --config workload (default: the configuration's)")
    ap.add_argument("--layers", type=int, default=0, help="truncate the stack (ncu captures of a small case only)")
    ap.add_argument("--oracle-rows", type=int, default=384, help="rows per sampled piece of the reference arm's bounded oracle step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the context measurements (full prefill, variants, first token)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_a3(args)


if __name__ == "__main__":
    main()
