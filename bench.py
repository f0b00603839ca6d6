#!/usr/bin/env python
"""Benchmark of the rectified MoE layer (arXiv 2402.12399) on B200.

One step = one pass of the whole hot path over one batch: rr_route (softmax/top-k,
capacity, Intra-GPU and Fill-in Rectification, tables) + rr_moe_fwd (gather, SwiGLU expert
FFN, combine) [+ rr_moe_bwd for the training workloads].  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c4|c5|c1] [--impl reference]

N > 1 runs N independent replicas (one process per GPU under torchrun); the layer has no
step that spans GPUs.  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2402_12399_b200 import synth  # noqa: E402

METRIC = "rectified MoE-layer tokens/s (route+FFN)"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return {"hbm_gbs": m["hbm_gbs"], "bf16_tflops": m["bf16_tflops"],
                "bf16_tflops_sustained": m["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            pass
    return local_rank


# ----------------------------------------------------------------------------------------
# inputs
# ----------------------------------------------------------------------------------------
def make_inputs(w: synth.Workload, cf_index: int, device):
    """Logits and hidden from the seeded host generator; the (large) expert weights are drawn on
    the device with a seeded torch generator: N(0, 0.02), bf16 (fp32 for c1)."""
    import torch
    seed = w.seed(cf_index)
    logits = synth.make_logits(w.T, w.E, w.bias, seed)
    rng = np.random.default_rng(seed + 7919)
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    hidden_h = torch.from_numpy(rng.standard_normal((w.T, w.d), dtype=np.float32)).to(tdt)
    g = torch.Generator(device=device)
    g.manual_seed(seed)

    def weight(*shape):
        t = torch.randn(*shape, generator=g, device=device, dtype=torch.float32)
        return t.mul_(0.02).to(tdt)

    W1, W3, W2 = weight(w.E, w.d_ff, w.d), weight(w.E, w.d_ff, w.d), weight(w.E, w.d, w.d_ff)
    dout = None
    if w.backward:
        dout = torch.randn(w.T, w.d, generator=g, device=device, dtype=torch.float32).to(tdt)
    return torch.from_numpy(logits), hidden_h, W1, W3, W2, dout


def to_host_bits(t):
    """torch tensor -> numpy array the oracle reads (float32, or uint16 bf16 bit patterns)."""
    import torch
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


# ----------------------------------------------------------------------------------------
# CPU oracle timing (the reported baseline and the --impl reference arm)
# ----------------------------------------------------------------------------------------
def oracle_step(orc, logits, hidden, W1, W3, W2, w, C, tokens):
    t0 = time.perf_counter()
    tab = orc.route(logits, w.k, C, w.G, w.mode)
    t1 = time.perf_counter()
    orc.forward_tokens(hidden, W1, W3, W2, logits, tab, tokens)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def oracle_throughput(w, t_route, t_fwd, n_tok):
    """tokens/s of the oracle: routing timed on all T tokens, the FFN on a token sample."""
    per_token = t_route / w.T + t_fwd / n_tok
    return 1.0 / per_token


def run_reference(args, w, cf_index, C):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    from oracle import rr_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    L = synth.make_layer(w.T, w.E, w.d, w.d_ff, w.bias, w.seed(cf_index), w.dtype, False) \
        if w.E * w.d * w.d_ff * 3 < (1 << 28) else None
    if L is None:   # full-size weights: only the experts' shapes matter for timing; draw them cheaply
        rng = np.random.default_rng(w.seed(cf_index))
        logits = synth.make_logits(w.T, w.E, w.bias, w.seed(cf_index))
        hidden = synth.to_bf16_bits(rng.standard_normal((w.T, w.d), dtype=np.float32))
        blk = synth.to_bf16_bits(rng.standard_normal((w.d_ff, w.d), dtype=np.float32) * np.float32(0.02))
        W1 = np.ascontiguousarray(np.broadcast_to(blk, (w.E, w.d_ff, w.d)))
        W3 = W1.copy()
        W2 = np.ascontiguousarray(W1.reshape(w.E, w.d, w.d_ff))
    else:
        logits, hidden, W1, W3, W2 = L.logits, L.hidden, L.W1, L.W3, L.W2
    cores = orc.num_threads()
    n_tok = max(1, cores)
    tokens = np.linspace(0, w.T - 1, n_tok).astype(np.int32)
    tr, tf = oracle_step(orc, logits, hidden, W1, W3, W2, w, C, tokens)   # calibration
    budget = 150.0 / max(1, args.steps + args.warmup)
    if tr + tf > budget and n_tok > 1:
        n_tok = max(1, int(n_tok * max(budget - tr, 0.05) / max(tf, 1e-9)))
        tokens = tokens[:n_tok]
    for _ in range(args.warmup):
        oracle_step(orc, logits, hidden, W1, W3, W2, w, C, tokens)
    t_route = t_fwd = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a, b = oracle_step(orc, logits, hidden, W1, W3, W2, w, C, tokens)
        t_route += a
        t_fwd += b
    wall = time.perf_counter() - t0
    value = oracle_throughput(w, t_route / args.steps, t_fwd / args.steps, n_tok)
    sample = f"routing on all {w.T} tokens + expert FFN/combine on {n_tok} tokens per step (forward only)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wall / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, cf_index, C),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(w, cf_index, C):
    return {"workload": w.name, "T": w.T, "E": w.E, "k": w.k, "G": w.G, "capacity": C,
            "capacity_factor": w.capacity_factors[cf_index], "d": w.d, "d_ff": w.d_ff,
            "mode": "IR+FR", "passes": "route+fwd+bwd" if w.backward else "route+fwd",
            "l2": "expert weights and activations exceed the 126 MB L2 many times over; no flush needed"}


# ----------------------------------------------------------------------------------------
# router-only measurement on the c2 workload (second half of the metric)
# ----------------------------------------------------------------------------------------
def time_router(rr, torch, logits_bufs, T, E, k, G, C, steps, warmup, one_graph=True, mode=3):
    """Median device time (us) of one rr_route call over the given logits buffers in rotation.
    `one_graph`: all buffers' calls are captured into a single CUDA graph (calls back to back, as
    inside a captured training or inference step) and a replay is divided by their number;
    otherwise one graph per call, so every call also pays a graph launch.  Returns (us, how)."""
    nbuf = len(logits_bufs)
    tab = rr.alloc_tables(T, E, k, C, G, mode)
    ws = rr.alloc_workspace(rr.route_workspace_bytes(T, E, k, C, G, mode))
    for i in range(warmup):
        rr.route(logits_bufs[i % nbuf], k, C, G, mode, tables=tab, workspace=ws)
    torch.cuda.synchronize()
    # the C-ABI call is capturable: no allocation, no synchronisation
    graphs = None
    try:
        graphs = []
        side = torch.cuda.Stream()
        groups = [logits_bufs] if one_graph else [[b] for b in logits_bufs]
        for grp in groups:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for b in grp:
                    rr.route(b, k, C, G, mode, tables=tab, workspace=ws)
            graphs.append(g)
        for g in graphs[:3]:
            g.replay()
        torch.cuda.synchronize()
    except Exception as exc:   # noqa: BLE001 - fall back to plain launches, say so in the output
        print(f"router: graph capture unavailable ({exc}); timing plain launches", file=sys.stderr)
        graphs = None
    per_launch = nbuf if (graphs and one_graph) else 1
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(steps):
        if graphs:
            graphs[i % len(graphs)].replay()
        else:
            rr.route(logits_bufs[i % nbuf], k, C, G, mode, tables=tab, workspace=ws)
        ev[i + 1].record()
    torch.cuda.synchronize()
    rr.check(ws)
    us = statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(steps)) * 1e3 / per_launch
    how = "plain stream launches" if not graphs else (
        f"cuda graph of {nbuf} calls of the C-ABI entry point, replayed" if one_graph else "one cuda graph per call, replayed")
    return us, how


def router_bytes(T, E, k, C):
    """Algorithmic bytes of one routing call: logits once + every table written once."""
    R = E * C + T
    return T * E * 4 + E * C * 5 + T * ((k + 1) * 8 + 16 + (k + 2) * 8) + 8 * R


def bench_router_shape(rr, torch, peaks, T, steps=20, warmup=3):
    """One router shape only (profiling aid): c2's experts, top-k, groups, bias and capacity factor 1.0
    on T tokens, default mode, rotating logits buffers larger than L2 together."""
    w = synth.WORKLOADS["c2"]
    C = T // w.E
    nbuf = max(2, -(-(300 << 20) // (T * w.E * 4)))
    base = torch.from_numpy(synth.make_logits(T, w.E, w.bias, w.seed(0) + 1)).cuda()
    bufs = [base] + [base.clone() for _ in range(nbuf - 1)]
    us, how = time_router(rr, torch, bufs, T, w.E, w.k, w.G, C, steps, warmup)
    alg = router_bytes(T, w.E, w.k, C)
    return {"T": T, "E": w.E, "k": w.k, "G": w.G, "capacity": C, "us_per_call": us, "algorithmic_bytes": alg,
            "achieved_gbs": alg / us / 1e3, "frac": alg / us / 1e3 / peaks["hbm_gbs"], "launch": how,
            "logits": f"{nbuf} rotating buffers (> L2)"}


def bench_router(rr, torch, peaks, steps=50, warmup=10):
    w = synth.WORKLOADS["c2"]
    C = w.capacity(1.0)
    nbuf = 20          # 20 x 16 MiB of logits > L2, rotated so every step reads HBM
    base = torch.from_numpy(synth.make_logits(w.T, w.E, w.bias, w.seed(0))).cuda()
    bufs = [base.clone() for _ in range(nbuf)]
    us, how = time_router(rr, torch, bufs, w.T, w.E, w.k, w.G, C, steps, warmup)
    us_single, _ = time_router(rr, torch, bufs, w.T, w.E, w.k, w.G, C, steps, warmup, one_graph=False)
    us_warm, _ = time_router(rr, torch, [bufs[0]] * nbuf, w.T, w.E, w.k, w.G, C, steps, warmup)   # logits stay in L2
    # the alternative readings of the paper's wording, same inputs and launch: score-priority dropping
    # (7 launches), the softmax-valued fill-in key (the persistent kernel with a second pass over each
    # row) and the capacity per source group (5 launches, G x E selection blocks)
    us_score, _ = time_router(rr, torch, bufs, w.T, w.E, w.k, w.G, C, steps, warmup, mode=3 | rr.SCORE)
    us_soft, _ = time_router(rr, torch, bufs, w.T, w.E, w.k, w.G, C, steps, warmup, mode=3 | rr.FR_SOFTMAX)
    us_local, _ = time_router(rr, torch, bufs, w.T, w.E, w.k, w.G, C, steps, warmup, mode=3 | rr.LOCAL_CAP)
    del bufs
    alg = router_bytes(w.T, w.E, w.k, C)
    gbs = alg / (us * 1e-6) / 1e9
    # the same router on sixteen times the tokens: how the rate grows once the fixed costs of the
    # five launches are spread over more data (not a substitute for c2)
    Tb = 1 << 20
    Cb = Tb // w.E
    big = [torch.from_numpy(synth.make_logits(Tb, w.E, w.bias, w.seed(0) + 1)).cuda()]
    big.append(big[0].clone())      # 2 x 256 MiB, each larger than L2
    us_big, _ = time_router(rr, torch, big, Tb, w.E, w.k, w.G, Cb, max(10, steps // 5), 3)
    del big
    torch.cuda.empty_cache()
    alg_big = router_bytes(Tb, w.E, w.k, Cb)
    return {"workload": "c2", "mode": "IR+FR", "capacity_factor": 1.0, "tokens_per_s": w.T / (us * 1e-6),
            "us_per_call": us, "algorithmic_bytes": alg, "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"],
            "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
            "kernels_per_call": "1 (persistent cooperative kernel; 7 / 5 launches with score-priority dropping / per-source capacity)",
            "launch": how, "logits": f"{nbuf} rotating buffers (> L2)",
            "one_graph_per_call": {"us_per_call": us_single, "achieved_gbs": alg / (us_single * 1e-6) / 1e9,
                                   "note": "every call also pays one graph launch"},
            "other_readings": {"score_priority_dropping_us_per_call": us_score, "softmax_fr_key_us_per_call": us_soft,
                               "per_source_capacity_us_per_call": us_local},
            "l2_warm": {"us_per_call": us_warm, "achieved_gbs": alg / (us_warm * 1e-6) / 1e9,
                        "logits": "one buffer, stays in L2"},
            "asymptote": {"T": Tb, "E": w.E, "k": w.k, "G": w.G, "capacity": Cb, "us_per_call": us_big,
                          "algorithmic_bytes": alg_big, "achieved_gbs": alg_big / (us_big * 1e-6) / 1e9,
                          "frac": alg_big / (us_big * 1e-6) / 1e9 / peaks["hbm_gbs"],
                          "tokens_per_s": Tb / (us_big * 1e-6)}}


def bench_aux(rr, torch, peaks, steps=30, warmup=5):
    """The load-balance loss (Section 5.1) and its gradient on the router shapes: c2 and sixteen times
    its tokens.  Calls are captured back to back into one CUDA graph over rotating logits buffers
    larger than L2 and a replay is divided by their number."""
    w = synth.WORKLOADS["c2"]
    res = []
    for T, nbuf in ((w.T, 20), (1 << 20, 2)):
        base = torch.from_numpy(synth.make_logits(T, w.E, w.bias, w.seed(0) + 2)).cuda()
        bufs = [base.clone() for _ in range(nbuf)]
        tab = rr.route(base, w.k, T * w.k // w.E, w.G, 3)
        ws = rr.alloc_workspace(rr.aux_workspace_bytes(T, w.E))
        dl = [torch.zeros(T, w.E, device="cuda") for _ in range(nbuf)]
        _, f, _ = rr.aux_loss_fwd(base, tab.topk_expert, 1e-2, workspace=ws)

        def timed(fn):
            for i in range(warmup):
                fn(i % nbuf)
            torch.cuda.synchronize()
            g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
            with torch.cuda.graph(g, stream=side):
                for i in range(nbuf):
                    fn(i)
            g.replay()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
            torch.cuda.synchronize()
            ev[0].record()
            for i in range(steps):
                g.replay()
                ev[i + 1].record()
            torch.cuda.synchronize()
            return statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(steps)) * 1e3 / nbuf

        us_f = timed(lambda i: rr.aux_loss_fwd(bufs[i], tab.topk_expert, 1e-2, workspace=ws))
        us_b = timed(lambda i: rr.aux_loss_bwd(bufs[i], f, 1e-2, 1.0, dlogits=dl[i]))
        # routing and the loss: two entry points that each read the logits, against rr_route_loss, whose
        # routing kernel adds the softmax values up in the pass it makes anyway
        Cq = T * w.k // w.E
        ws_r = rr.alloc_workspace(rr.route_workspace_bytes(T, w.E, w.k, Cq, w.G, 3))
        ws_l = rr.alloc_workspace(rr.route_loss_workspace_bytes(T, w.E, w.k, Cq, w.G, 3))
        aux_out = tuple(torch.empty(n, device="cuda") for n in (1, w.E, w.E))

        def two_calls(i):
            rr.route(bufs[i], w.k, Cq, w.G, 3, tables=tab, workspace=ws_r)
            rr.aux_loss_fwd(bufs[i], tab.topk_expert, 1e-2, workspace=ws)

        us_two = timed(two_calls)
        us_one = timed(lambda i: rr.route_loss(bufs[i], w.k, Cq, w.G, 3, 1e-2, tables=tab, workspace=ws_l, aux=aux_out))
        rr.check(ws_r); rr.check(ws_l)
        us_a = timed(lambda i: rr.aux_loss_bwd(bufs[i], f, 1e-2, 1.0, dlogits=dl[i], accumulate=True))
        rr.check(ws)
        bytes_f = T * w.E * 4 + T * 4            # logits once + the first choices
        bytes_b = 2 * T * w.E * 4                # logits once, gradient written once (read too when added)
        res.append({"T": T, "E": w.E, "fwd_us": us_f, "fwd_gbs": bytes_f / us_f / 1e3,
                    "fwd_frac": bytes_f / us_f / 1e3 / peaks["hbm_gbs"], "fwd_algorithmic_bytes": bytes_f,
                    "bwd_us": us_b, "bwd_gbs": bytes_b / us_b / 1e3, "bwd_frac": bytes_b / us_b / 1e3 / peaks["hbm_gbs"],
                    "bwd_algorithmic_bytes": bytes_b, "bwd_accumulate_us": us_a,
                    "bwd_accumulate_gbs": 3 * T * w.E * 4 / us_a / 1e3,
                    "route+aux_loss_fwd_us": us_two, "route_loss_us": us_one,
                    "logits": f"{nbuf} rotating buffers (> L2)"})
        del bufs, dl, base
        torch.cuda.empty_cache()
    return {"bound": "hbm", "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "kernels_per_call": "2 fwd (+1 memset), 1 bwd",
            "launch": "cuda graph of all buffers' calls, replayed", "shapes": res}


def bench_gate(rr, torch, peaks, steps=30, warmup=5):
    """The gate projection logits = hidden . Wg^T (Eq. 1) and its backward on the c3 and c5 shapes.
    The forward is bound by the one read of `hidden`; rotating inputs larger than L2."""
    res = []
    for name in ("c3", "c5"):
        w = synth.WORKLOADS[name]
        T, E, d = w.T, w.E, w.d
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed(0))
        nbuf = 3     # 3 x 128 MiB of hidden states > L2
        hid = [torch.randn(T, d, generator=g, device="cuda").to(torch.bfloat16) for _ in range(nbuf)]
        Wg = (torch.randn(E, d, generator=g, device="cuda") / d ** 0.5).to(torch.bfloat16)
        fwd_b, bwd_b = rr.gate_workspace_bytes(T, E, d)
        ws_f, ws_b = rr.alloc_workspace(fwd_b), rr.alloc_workspace(bwd_b)
        logits = torch.empty(T, E, device="cuda")
        dl = torch.randn(T, E, generator=g, device="cuda")
        dh = torch.zeros(T, d, device="cuda")
        dW = torch.empty(E, d, device="cuda")

        def timed(fn):
            for i in range(warmup):
                fn(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for i in range(steps):
                fn(i)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / steps * 1e3

        us_f = timed(lambda i: rr.gate_fwd(hid[i % nbuf], Wg, logits=logits, workspace=ws_f))
        us_b = timed(lambda i: rr.gate_bwd(dl, hid[i % nbuf], Wg, dh, dWg=dW, workspace=ws_b))
        rr.check(ws_f)
        # projection + routing + load-balance loss: three entry points (4 launches and a memset) against
        # rr_gate_route (2 launches, the selection in the projection's epilogue, logits never read back)
        C = w.capacity(1.0)
        tab = rr.alloc_tables(T, E, w.k, C, w.G, 3)
        ws_r = rr.alloc_workspace(rr.route_workspace_bytes(T, E, w.k, C, w.G, 3))
        ws_a = rr.alloc_workspace(rr.aux_workspace_bytes(T, E))
        ws_g = rr.alloc_workspace(rr.gate_route_workspace_bytes(T, E, w.k, C, w.G, 3, d))
        aux_out = tuple(torch.empty(n, device="cuda") for n in (1, E, E))

        def separate(i):
            rr.gate_fwd(hid[i % nbuf], Wg, logits=logits, workspace=ws_f)
            rr.route(logits, w.k, C, w.G, 3, tables=tab, workspace=ws_r)
            rr.aux_loss_fwd(logits, tab.topk_expert, 1e-2, workspace=ws_a)

        def graphed(fn):
            """device time per call: the calls on all input buffers captured into one graph, replayed"""
            for i in range(warmup):
                fn(i)
            torch.cuda.synchronize()
            g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
            with torch.cuda.graph(g, stream=side):
                for i in range(nbuf):
                    fn(i)
            g.replay()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
            torch.cuda.synchronize()
            ev[0].record()
            for i in range(steps):
                g.replay()
                ev[i + 1].record()
            torch.cuda.synchronize()
            return statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(steps)) * 1e3 / nbuf

        us_sep = graphed(separate)
        us_fused = graphed(lambda i: rr.gate_route(hid[i % nbuf], Wg, w.k, C, w.G, 3, 1e-2, logits=logits, tables=tab,
                                                   workspace=ws_g, aux=aux_out))
        us_f_graph = graphed(lambda i: rr.gate_fwd(hid[i % nbuf], Wg, logits=logits, workspace=ws_f))

        def separate_no_loss(i):
            rr.gate_fwd(hid[i % nbuf], Wg, logits=logits, workspace=ws_f)
            rr.route(logits, w.k, C, w.G, 3, tables=tab, workspace=ws_r)

        us_sep0 = graphed(separate_no_loss)
        us_fused0 = graphed(lambda i: rr.gate_route(hid[i % nbuf], Wg, w.k, C, w.G, 3, None, logits=logits, tables=tab,
                                                    workspace=ws_g))
        rr.check(ws_r); rr.check(ws_g)
        bytes_f = T * d * 2 + E * d * 2 + T * E * 4
        bytes_b = T * d * 2 + 2 * T * d * 4 + T * E * 4 * 2 + E * d * (2 + 4)   # hidden, dhidden read+write, dlogits twice
        res.append({"shape": name, "T": T, "E": E, "d": d, "dtype": "bf16",
                    "fwd_us": us_f, "fwd_gbs": bytes_f / (us_f * 1e-6) / 1e9, "fwd_frac": bytes_f / (us_f * 1e-6) / 1e9 / peaks["hbm_gbs"],
                    "fwd_algorithmic_bytes": bytes_f, "fwd_tflops": 2.0 * T * E * d / (us_f * 1e-6) / 1e12,
                    "bwd_us": us_b, "bwd_gbs": bytes_b / (us_b * 1e-6) / 1e9, "bwd_frac": bytes_b / (us_b * 1e-6) / 1e9 / peaks["hbm_gbs"],
                    "bwd_algorithmic_bytes": bytes_b,
                    "graph_replay_us": {"gate_fwd": us_f_graph, "gate_fwd+route+aux_loss_fwd": us_sep, "gate_route": us_fused,
                                        "gate_fwd+route": us_sep0, "gate_route_without_loss": us_fused0}})
        del hid, dh
        torch.cuda.empty_cache()
    return {"bound": "hbm", "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
            "inputs": "3 rotating hidden buffers (> L2)", "shapes": res}


# The capacity sweeps of the paper's Tables 3 and 4 on the c3 layer: (k, capacity factor, mode); the
# capacity factor already contains k (Section 3), mode bit 0 = IR, bit 1 = FR
SWEEP = [(1, 1.0, 0), (1, 1.0, 3), (1, 0.75, 0), (1, 0.75, 1), (1, 0.5, 0), (1, 0.5, 1),
         (1, 1.25, 0), (1, 1.25, 2), (1, 1.5, 0), (1, 1.5, 2),
         (2, 2.0, 0), (2, 2.0, 3), (2, 1.5, 0), (2, 1.5, 1), (2, 1.0, 0), (2, 1.0, 1),
         (2, 2.5, 0), (2, 2.5, 2), (2, 3.0, 0), (2, 3.0, 2)]


def bench_sweep(rr, torch, steps=10, warmup=3):
    """Forward pass (route + FFN) of the c3 layer under the routers and capacity factors of the
    paper's inference sweeps; one set of weights, the capacity and the mode vary."""
    w = synth.WORKLOADS["c3"]
    device = torch.device("cuda", torch.cuda.current_device())
    logits_h, hidden_h, W1, W3, W2, _ = make_inputs(w, 0, device)
    logits, hidden = logits_h.to(device), hidden_h.to(device)
    dt = rr.binding._dtype_code(hidden)
    out = torch.empty(w.T, w.d, dtype=torch.float32, device=device)
    rows_out = []
    for k, cf, mode in SWEEP:
        C = int(cf * w.T / w.E)
        tab = rr.alloc_tables(w.T, w.E, k, C, w.G, mode, device)
        ws_r = rr.alloc_workspace(rr.route_workspace_bytes(w.T, w.E, k, C, w.G, mode), device)
        ws_f = rr.alloc_workspace(rr.moe_workspace_bytes(w.T, w.E, k, C, w.G, w.d, w.d_ff, dt, mode)[0], device)

        def step():
            rr.route(logits, k, C, w.G, mode, tables=tab, workspace=ws_r)
            rr.moe_fwd(hidden, W1, W3, W2, logits, tab, out=out, workspace=ws_f)

        for _ in range(warmup):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        rr.check(ws_r); rr.check(ws_f)
        ms = e0.elapsed_time(e1) / steps
        dropped = int((tab.drop_count > 0).sum().item())
        rows_out.append({"k": k, "capacity_factor": cf, "capacity": C,
                         "router": "top-%d%s%s" % (k, "+FR" if mode & 2 else "", "+IR" if mode & 1 else ""),
                         "live_rows": int(tab.row_offset[-1].item()), "tokens_with_a_drop": dropped,
                         "ms_per_step": ms, "tokens_per_s": w.T / (ms * 1e-3)})
        del tab, ws_r, ws_f
    return {"workload": "c3 layer (T=16384, E=8, G=4, d=4096, d_ff=14336), forward", "steps": steps, "sweep": rows_out}


# ----------------------------------------------------------------------------------------
def matmul_on_this_box(torch, device, seconds=1.5):
    """Sustained rate of the library's bf16 matmul (8192^3, back to back) on the GPU this run got: context for
    `roofline.frac`, whose denominator was measured on another GPU of the pool (their power caps differ)."""
    n = 8192
    a = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    b = torch.randn(n, n, device=device, dtype=torch.bfloat16)
    c = torch.empty(n, n, device=device, dtype=torch.bfloat16)
    for _ in range(5):
        torch.matmul(a, b, out=c)
    torch.cuda.synchronize()
    reps = 200
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total_ms, total_n = 0.0, 0
    while total_ms < seconds * 1e3:
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        total_ms, total_n = total_ms + ms, total_n + reps
        last = 2.0 * n ** 3 * reps / (ms * 1e-3) / 1e12
    del a, b, c
    return {"tflops": last, "tflops_whole_loop": 2.0 * n ** 3 * total_n / (total_ms * 1e-3) / 1e12,
            "how": f"torch.matmul bf16 {n}^3 back to back for {total_ms / 1e3:.1f} s; the last {reps} calls"}


def reduce_max_ms(torch, dist, ms, world, device):
    """The slowest rank's time: every rank ends up with the maximum over the job."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world, tokens_per_rank, ms_step):
    """Replicas: every rank pushes its own batch through its own layer; the job's rate is the sum."""
    return world * tokens_per_rank / (ms_step * 1e-3)


def shrink(w: synth.Workload, n: int) -> synth.Workload:
    """Same per-expert problem with T, E and G divided by n (profiling aid: every kernel keeps its
    tile shapes and per-expert row counts while the footprint and the traffic scale by 1/n)."""
    if n <= 1:
        return w
    assert w.T % n == 0 and w.E % n == 0 and w.G % n == 0, "shrink factor must divide T, E and G"
    return synth.Workload(f"{w.name}/{n}", w.T // n, w.E // n, w.k, w.G // n, w.capacity_factors, w.bias, w.d,
                          w.d_ff, w.dtype, w.backward, w.mode, w.index)


def measure(rr, torch, dist, w, cf_index, steps, warmup, world, local_rank, device, peaks, backward, want_e2e):
    """Times `steps` passes of the hot path on one workload; returns the measurements."""
    C = w.capacity(w.capacity_factors[cf_index])
    logits_h, hidden_h, W1, W3, W2, dout = make_inputs(w, cf_index, device)
    logits_h, hidden_h = logits_h.pin_memory(), hidden_h.pin_memory()
    logits, hidden = logits_h.to(device), hidden_h.to(device)
    dt = rr.binding._dtype_code(hidden)
    tab = rr.alloc_tables(w.T, w.E, w.k, C, w.G, w.mode, device)
    ws_route = rr.alloc_workspace(rr.route_workspace_bytes(w.T, w.E, w.k, C, w.G, w.mode), device)
    fwd_b, bwd_b, saved_b = rr.moe_workspace_bytes(w.T, w.E, w.k, C, w.G, w.d, w.d_ff, dt, w.mode)
    ws_fwd = rr.alloc_workspace(fwd_b, device)
    out = torch.empty(w.T, w.d, dtype=torch.float32, device=device)
    saved = ws_bwd = grads = None
    if backward:
        saved = torch.empty(saved_b, dtype=torch.uint8, device=device)
        ws_bwd = rr.alloc_workspace(bwd_b, device)
        f32 = dict(dtype=torch.float32, device=device)
        grads = (torch.empty(w.T, w.d, **f32), torch.empty(w.T, w.E, **f32), torch.empty(w.E, w.d_ff, w.d, **f32),
                 torch.empty(w.E, w.d_ff, w.d, **f32), torch.empty(w.E, w.d, w.d_ff, **f32))

    def step(trace_f=None, trace_b=None):
        rr.route(logits, w.k, C, w.G, w.mode, tables=tab, workspace=ws_route)
        rr.moe_fwd(hidden, W1, W3, W2, logits, tab, out=out, saved=saved, workspace=ws_fwd, trace=trace_f)
        if backward:
            rr.moe_bwd(dout, hidden, W1, W3, W2, logits, tab, saved, workspace=ws_bwd, grads=grads, trace=trace_b)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return reduce_max_ms(torch, dist, ms, world, device)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    rr.check(ws_route); rr.check(ws_fwd)
    if backward:
        rr.check(ws_bwd)
    rows = int(tab.row_offset[-1].item())

    traces_f = [rr.Trace() for _ in range(steps)]
    traces_b = [rr.Trace() for _ in range(steps)] if backward else [None] * steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(visible_gpu_index(local_rank))
    barrier()
    sampler.start()
    e0.record()
    for i in range(steps):
        step(traces_f[i], traces_b[i])
    e1.record()
    barrier()
    clocks = sampler.stop()
    rr.check(ws_fwd)
    ms_step = max_over_ranks(e0.elapsed_time(e1)) / steps

    # per-kernel times from the events the library records around its launches; the dominant
    # kernel (largest share of the step) carries the roofline entry
    dF = float(w.d) * w.d_ff * rows
    kern = {"gate_up_gemm": (statistics.mean(tr.ms(0, 1) for tr in traces_f), 4.0 * dF),
            "down_gemm": (statistics.mean(tr.ms(1, 2) for tr in traces_f), 2.0 * dF)}
    if backward:
        kern["dact_gemm"] = (statistics.mean(tr.ms(0, 1) for tr in traces_b), 2.0 * dF)
        kern["dx_gemm"] = (statistics.mean(tr.ms(1, 2) for tr in traces_b), 4.0 * dF)
        kern["wgrad_gemms_x3"] = (statistics.mean(tr.ms(2, 3) for tr in traces_b), 6.0 * dF)
    peak_tf = peaks["bf16_tflops_sustained"] * (0.5 if w.dtype == "f32" else 1.0)
    mhz = clocks.get("sm_mhz") or 0.0
    # Bytes each kernel has to move through HBM at least once: its row-indexed operands and results (live
    # rows), every expert's weights once, the token-indexed fp32 result of the combine kernels once.  The
    # short-K training shapes are bound by these, not by the tensor cores (g and u are kept in fp32).
    es = 4 if w.dtype == "f32" else 2
    RF, RD, WT = float(rows) * w.d_ff, float(rows) * w.d, float(w.E) * w.d * w.d_ff
    hbm = {"gate_up_gemm": RD * es + 2 * WT * es + RF * es + (RF * 8 if backward else 0),
           "down_gemm": RF * es + WT * es + float(w.T) * w.d * 4,
           "dact_gemm": RD * 2 + WT * 2 + RF * 8 + 3 * RF * 2,
           "dx_gemm": 2 * RF * 2 + 2 * WT * 2 + float(w.T) * w.d * 4,
           "wgrad_gemms_x3": 3 * (RD + RF) * 2 + 3 * WT * 4}
    # time x median SM clock: what the kernel costs in cycles, whatever the power cap did to the clock
    kernels = {n: {"ms_per_step": ms, "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_peak": fl / (ms * 1e-3) / 1e12 / peak_tf,
                   "hbm_bytes": hbm[n], "hbm_gbs": hbm[n] / (ms * 1e-3) / 1e9,
                   "hbm_frac": hbm[n] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                   "mcycles_per_step": ms * mhz * 1e-3, "flops_per_cycle": (fl / (ms * mhz * 1e3)) if mhz else None}
               for n, (ms, fl) in kern.items()}
    for v in kernels.values():
        v["bound"] = "hbm" if v["hbm_frac"] > v["frac_of_peak"] else "tensor"
    dom = max(kern, key=lambda n: kern[n][0])
    dom_ms, dom_fl = kern[dom]
    launches_in_dom = 3 if dom == "wgrad_gemms_x3" else 1
    achieved = dom_fl / (dom_ms * 1e-3) / 1e12
    tot_fl, tot_ms = sum(f for _, f in kern.values()), sum(m for m, _ in kern.values())
    # DRAM bytes of one gate/up launch on the full c3 workload: ncu counters taken on c3 with T and E
    # halved (2.47 GB read + written), times two because the traffic follows the number of experts
    traffic = 4.94e9 if (w.name == "c3" and dom == "gate_up_gemm") else None
    roofline = {"bound": "tensor", "kernel": f"k_gemm<{dom}>", "achieved": achieved, "peak": peak_tf,
                "unit": "TFLOP/s", "frac": achieved / peak_tf, "traffic": traffic,
                "peak_source": f"{peaks['source']} sustained bf16 matmul" + (" x 0.5 (tf32)" if w.dtype == "f32" else ""),
                "flops_per_launch": dom_fl / launches_in_dom, "live_rows": rows,
                "ms_per_launch": dom_ms / launches_in_dom, "kernels": kernels,
                "all_gemms": {"tflops": tot_fl / (tot_ms * 1e-3) / 1e12,
                              "frac_of_peak": tot_fl / (tot_ms * 1e-3) / 1e12 / peak_tf, "ms_per_step": tot_ms}}

    res = {"C": C, "ms_step": ms_step, "value": whole_job_tokens_per_s(world, w.T, ms_step), "clocks": clocks, "roofline": roofline,
           "rows": rows, "launches_per_step": 1 + 4 + (8 if backward else 0),
           "host": (logits_h, hidden_h, W1, W3, W2)}

    if want_e2e:
        # Inputs come from pinned host memory every step and the result is read back every step.
        # Two sets of device buffers and three streams: the upload of step i+1 and the read-back of
        # step i-1 run beside the kernels of step i, as a caller who streams batches would arrange it.
        out_h = [torch.empty(w.T, w.d, dtype=torch.float32).pin_memory() for _ in range(2)]
        lg2, hd2, out2 = [logits, torch.empty_like(logits)], [hidden, torch.empty_like(hidden)], [out, torch.empty_like(out)]
        s_in, s_out, s_cmp = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device), torch.cuda.current_stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        e2e_steps = max(3, min(steps, 20))
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def e2e_step(i):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[b])       # the kernels that read this input set are done
                lg2[b].copy_(logits_h, non_blocking=True)
                hd2[b].copy_(hidden_h, non_blocking=True)
                ev_in[b].record(s_in)
            s_cmp.wait_event(ev_in[b])
            if i >= 2:
                s_cmp.wait_event(ev_out[b])          # the previous result in this output set has been read
            rr.route(lg2[b], w.k, C, w.G, w.mode, tables=tab, workspace=ws_route)
            rr.moe_fwd(hd2[b], W1, W3, W2, lg2[b], tab, out=out2[b], saved=saved, workspace=ws_fwd)
            if backward:
                rr.moe_bwd(dout, hd2[b], W1, W3, W2, lg2[b], tab, saved, workspace=ws_bwd, grads=grads)
            ev_cmp[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[b])
                out_h[b].copy_(out2[b], non_blocking=True)
                ev_out[b].record(s_out)

        def drain():
            for b in range(2):
                s_cmp.wait_event(ev_out[b])

        for i in range(4):
            e2e_step(i)
        drain()
        barrier()
        a0.record()
        for i in range(e2e_steps):
            e2e_step(i + 4)
        drain()                                      # the last read-backs are inside the timed region
        a1.record()
        barrier()
        rr.check(ws_fwd)
        e2e_ms = max_over_ranks(a0.elapsed_time(a1)) / e2e_steps
        h2d = logits_h.numel() * 4 + hidden_h.numel() * hidden_h.element_size()
        res["e2e"] = {"value": whole_job_tokens_per_s(world, w.T, e2e_ms), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": out_h[0].numel() * 4, "ms_per_step": e2e_ms, "steps": e2e_steps,
                      "overlap": "two buffer sets, copies of neighbouring steps run beside the kernels",
                      "read_back": "the layer output out[T,d] fp32 only; the routing tables stay on the device, where "
                                   "rr_moe_fwd / rr_moe_bwd consume them"}
    return res


def relaunch_under_torchrun(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one process per GPU, replicas of
    the layer) under torch.distributed.run on this node and hand back its exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--cf-index", type=int, default=0)
    ap.add_argument("--forward-only", action="store_true", help="skip rr_moe_bwd on the training workloads")
    ap.add_argument("--shrink", type=int, default=1, help="divide T, E and G by this factor (profiling aid)")
    ap.add_argument("--no-router", action="store_true", help="skip the router-only c2 and the gate projection measurements")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-training", action="store_true", help="skip the short c4 training-step measurement")
    ap.add_argument("--gate", action="store_true", help="only the gate projection measurement (prints its JSON object)")
    ap.add_argument("--aux", action="store_true", help="only the load-balance loss measurement (prints its JSON object)")
    ap.add_argument("--sweep", action="store_true",
                    help="only the capacity-factor sweeps of the paper's Tables 3-4 on the c3 layer (prints their JSON object)")
    ap.add_argument("--router-only", action="store_true",
                    help="only the router measurement on c2 (prints its JSON object); used for profiling")
    ap.add_argument("--router-tokens", type=int, default=0,
                    help="with --router-only: time just the default mode on this many tokens (c2's other parameters)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = shrink(synth.WORKLOADS[args.workload], args.shrink)
    if w.d == 0:
        raise SystemExit("c2 is the router-only workload; it is reported inside every line as 'router'")
    C = w.capacity(w.capacity_factors[args.cf_index])

    if args.impl == "reference":
        if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
            raise SystemExit(relaunch_under_torchrun(args.gpus))
        run_reference(args, w, args.cf_index, C)
        return
    if args.gate:
        import torch
        import paper_2402_12399_b200 as rr
        print(json.dumps(bench_gate(rr, torch, measured_peaks(), steps=min(args.steps, 30), warmup=args.warmup)))
        return
    if args.aux:
        import torch
        import paper_2402_12399_b200 as rr
        print(json.dumps(bench_aux(rr, torch, measured_peaks())))
        return
    if args.sweep:
        import torch
        import paper_2402_12399_b200 as rr
        print(json.dumps(bench_sweep(rr, torch, steps=min(args.steps, 20))))
        return
    if args.router_only:
        import torch
        import paper_2402_12399_b200 as rr
        if args.router_tokens:
            print(json.dumps(bench_router_shape(rr, torch, measured_peaks(), args.router_tokens, steps=args.steps,
                                                warmup=args.warmup)))
        else:
            print(json.dumps(bench_router(rr, torch, measured_peaks(), steps=args.steps, warmup=args.warmup)))
        return

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(relaunch_under_torchrun(args.gpus))

    import torch
    import torch.distributed as dist
    import paper_2402_12399_b200 as rr
    rr.lib()   # fail loudly if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    peaks = measured_peaks()
    backward = w.backward and not args.forward_only

    m = measure(rr, torch, dist, w, args.cf_index, args.steps, args.warmup, world, local_rank, device, peaks,
                backward, want_e2e=True)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if world == 1 and not args.no_cpu:
        from oracle import rr_oracle as orc
        logits_h, hidden_h, W1, W3, W2 = m["host"]
        cores = orc.num_threads()
        lg, hd = logits_h.numpy(), to_host_bits(hidden_h)
        w1, w3, w2 = to_host_bits(W1), to_host_bits(W3), to_host_bits(W2)
        n_tok = cores
        tokens = np.linspace(0, w.T - 1, n_tok).astype(np.int32)
        tr_, tf_ = oracle_step(orc, lg, hd, w1, w3, w2, w, C, tokens)
        if tf_ < 8.0:       # grow the sample towards ~15 s of CPU work
            n_tok = int(min(w.T, max(n_tok, n_tok * 15.0 / max(tf_, 1e-3))))
            tokens = np.linspace(0, w.T - 1, n_tok).astype(np.int32)
            tr_, tf_ = oracle_step(orc, lg, hd, w1, w3, w2, w, C, tokens)
        cpu = {"value": oracle_throughput(w, tr_, tf_, n_tok), "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": f"routing on all {w.T} tokens ({tr_:.2f} s) + expert FFN/combine on {n_tok} evenly spaced "
                         f"tokens ({tf_:.2f} s), forward only"}
        del w1, w3, w2
    m.pop("host")
    torch.cuda.empty_cache()

    router = None if args.no_router or world > 1 else bench_router(rr, torch, peaks)
    gate = None if args.no_router or world > 1 else bench_gate(rr, torch, peaks, steps=10, warmup=3)
    aux = None if args.no_router or world > 1 else bench_aux(rr, torch, peaks, steps=10, warmup=3)

    training = None
    if not args.no_training and world == 1 and not w.backward:
        # the backward rows of the hot path on the two training workloads, briefly
        training = []
        for name in ("c4", "c5"):
            wt = synth.WORKLOADS[name]
            tm = measure(rr, torch, dist, wt, 0, max(20, args.steps // 2), 3, 1, local_rank, device, peaks, True, False)
            tm.pop("host")
            training.append({"workload": name, "passes": "route+fwd+bwd", "capacity_factor": 1.0, "tokens_per_s": tm["value"],
                             "ms_per_step": tm["ms_step"], "live_rows": tm["rows"], "kernels": tm["roofline"]["kernels"],
                             "all_gemms": tm["roofline"]["all_gemms"], "clocks": tm["clocks"]})
            del tm
            torch.cuda.empty_cache()

    latency = None
    if not args.no_training and world == 1 and w.name != "c1":
        # the small parity workload (fp32 inputs as tf32): no roofline claim, a step is launch- and host-bound
        w1 = synth.WORKLOADS["c1"]
        t1 = measure(rr, torch, dist, w1, 0, 50, 5, 1, local_rank, device, peaks, False, False)
        t1.pop("host")
        latency = {"workload": "c1", "passes": "route+fwd", "ms_per_step": t1["ms_step"], "tokens_per_s": t1["value"],
                   "live_rows": t1["rows"], "note": "stream launches from Python, one after the other; 5 kernels and a memset per step"}
        del t1

    if world == 1 and not args.no_cpu and w.dtype != "f32":
        ref = matmul_on_this_box(torch, device)
        ref["achieved_over_it"] = m["roofline"]["achieved"] / ref["tflops"]
        m["roofline"]["matmul_on_this_box"] = ref
    cfg = config_dict(w, args.cf_index, C)
    cfg["passes"] = "route+fwd+bwd" if backward else "route+fwd"
    line = {"metric": METRIC, "value": m["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": m["ms_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "tf32" if w.dtype == "f32" else "bf16", "data": "synthetic",
            "config": cfg, "clocks": m["clocks"], "e2e": m["e2e"],
            "gpu_launches": m["launches_per_step"] * args.steps, "roofline": m["roofline"], "cpu_baseline": cpu,
            "router": router, "gate": gate, "aux_loss": aux, "latency_c1": latency, "training": training}
    if router is not None:
        # the second half of the metric once more, compact and last in the line
        line["router_c2"] = {"us_per_call": router["us_per_call"], "tokens_per_s": router["tokens_per_s"],
                             "achieved_gbs": router["achieved_gbs"], "peak_gbs": router["peak_gbs"], "frac": router["frac"],
                             "asymptote_T": router["asymptote"]["T"], "asymptote_us_per_call": router["asymptote"]["us_per_call"],
                             "asymptote_frac": router["asymptote"]["frac"]}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
