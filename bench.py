#!/usr/bin/env python
"""Benchmark of the packed verify step (allocation -> attention x L -> acceptance).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic
input, replayed as ONE captured CUDA graph.  The default workload is the
Qwen3-8B-shaped full step at concurrency 32 (36 layers, contexts 2048-8192).
Beside the headline (K replays between two barriers) the line carries the per-replay median and
minimum, a sustained leg (seconds of replays, clock settled under the power cap), the attention
kernel's roofline at both, the whole decision chain as one graph, and the CPU oracle's time.
Prints one JSON line (rank 0).  With N > 1 (launched by torch.distributed.run)
every rank runs an independent replica on its own GPU with its own batch:
the path shards by request and needs no collective, so scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from dscale_inputs import (CONFIGS, make_kv_layer, make_lm_head_unpacked, make_logits_unpacked,  # noqa: E402
                           make_predictor_inputs, make_q_unpacked, make_requests, rows_to_packed, small_variant)

SCALE = 1.0 / float(np.sqrt(128.0))
METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
FLUSH_BYTES = 384 * 1024 * 1024          # rewritten between replays of a step that fits the L2


# --------------------------------------------------------------------- helpers
def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def measured_bf16_peak():
    """Dense bf16 tensor peak in TFLOP/s for a kernel timed alone (burst figure)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["bf16_tflops"])
        except Exception:
            pass
    return 1590.0


def recorded_traffic(workload: str):
    """DRAM bytes per attention launch from the committed ncu summary, if any."""
    p = os.path.join(ROOT, "profiles", "attn_tc_traffic.json")
    if os.path.exists(p):
        try:
            return json.load(open(p)).get(workload)
        except Exception:
            return None
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def algorithmic_bytes(cfg, req, k):
    """Bytes the method must move: per layer K and V of every visible key, the
    page ids, Q in and O out; per step the logits, scores and packed fields."""
    n = req["n_live"]
    kv_len = req["ctx_len"][:n].astype(np.int64) + np.asarray(k[:n], dtype=np.int64)
    kv = int(kv_len.sum()) * cfg.n_kv_heads * 128 * 2 * 2
    pages = int(((kv_len + 15) // 16).sum()) * 4
    qo = 2 * 8 * n * cfg.n_q_heads * 128 * 2
    per_layer = kv + pages + qo
    logits = 8 * n * cfg.vocab * 4
    small = n * 15 * 4 + n * 16 * 4 + 4 * 8 * n * 4 + n * 19 * 4
    return per_layer, logits + small


def step_bytes_of(cfg, req):
    """Algorithmic bytes of one step; needs no allocation (the lengths sum to 8 N)."""
    n = req["n_live"]
    kv_tok = int(req["ctx_len"][:n].astype(np.int64).sum()) + 8 * n
    pages = int(((req["ctx_len"][:n].astype(np.int64) + 8 + 15) // 16).sum())     # about: lengths vary around 8
    per_layer = kv_tok * cfg.n_kv_heads * 128 * 2 * 2 + pages * 4 + 2 * 8 * n * cfg.n_q_heads * 128 * 2
    return per_layer * cfg.layers + 8 * n * cfg.vocab * 4


def workload_config(cfg, req, attn="tensor"):
    """The `config` object of the JSON line: the same for both arms (the reference arm times the
    CPU oracle on a sample of exactly this workload)."""
    n = req["n_live"]
    sb = step_bytes_of(cfg, req)
    flush = sb < 4 * L2_BYTES
    return {"workload": cfg.name, "requests_per_gpu": n, "layers": cfg.layers,
            "heads": [cfg.n_q_heads, cfg.n_kv_heads], "ctx": [cfg.ctx_lo, cfg.ctx_hi],
            "vocab": cfg.vocab, "packed_rows": 8 * n, "attn": attn,
            "l2": ("inputs_larger_than_L2 (%.1f GB per step)" % (sb / 1e9)) if not flush else
                  ("L2 flushed before every timed replay (a %d MB buffer rewritten; %.1f MB per step); "
                   "step time = sum of the per-replay intervals" % (FLUSH_BYTES >> 20, sb / 1e6)),
            "launch": "one captured CUDA graph per step"}


# ------------------------------------------------------------------ CPU oracle
def oracle_step_sample(cfg, req, kvs, q_unpacked, logits_unpacked):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload:
    allocation and acceptance in full, attention on the first len(kvs) layers
    (all requests), and scales the attention time to cfg.layers layers.
    Returns (tokens_per_s, seconds of CPU work, description)."""
    from oracle import accept as OC
    from oracle import dvl_alloc as OA
    from oracle import verify_attn as OV
    t0 = time.perf_counter()
    alloc = OA.dvl_alloc(req["n_bs"], req["n_live"], req["scores"], req["draft_tokens"],
                         req["ctx_len"], req["block_table"])
    t_alloc = time.perf_counter() - t0
    lp = rows_to_packed(logits_unpacked, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"])
    lf = lp.numpy()
    t_attn = 0.0
    for (kc, vc), qu in zip(kvs, q_unpacked):
        qp = rows_to_packed(qu, alloc["k"], alloc["offset"], req["n_live"], 8 * req["n_bs"])
        qf, kf, vf = qp.float().numpy(), kc.float().numpy(), vc.float().numpy()
        t2 = time.perf_counter()
        OV.verify_attn(qf, kf, vf, req["block_table"], req["ctx_len"], alloc["k"], alloc["offset"],
                       req["n_live"], cfg.n_q_heads, cfg.n_kv_heads, SCALE)
        t_attn += time.perf_counter() - t2
    t3 = time.perf_counter()
    res = OC.accept(lf, cfg.vocab, alloc["tokens"], alloc["k"], alloc["offset"], req["n_live"],
                    req["n_bs"])
    t_acc = time.perf_counter() - t3
    tokens = int(res["out_len"].sum())
    step = t_alloc + cfg.layers * (t_attn / len(kvs)) + t_acc
    work = t_alloc + t_attn + t_acc
    desc = (f"allocation and acceptance in full, attention on the first {len(kvs)} of {cfg.layers} "
            f"layers (all {req['n_live']} requests), attention time scaled to {cfg.layers} layers")
    return tokens / step, work, desc


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, rank):
    """Reference arm: the CPU oracle timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    cfg = CONFIGS[args.workload]
    req = make_requests(cfg)
    n_l = min(cfg.layers, args.cpu_layers)
    kvs = [make_kv_layer(req, l, poison=False) for l in range(n_l)]
    qus = [make_q_unpacked(req, l) for l in range(n_l)]
    lu = make_logits_unpacked(req)
    vals, work = [], 0.0
    desc = ""
    for s in range(args.warmup + args.steps):
        v, w, desc = oracle_step_sample(cfg, req, kvs, qus, lu)
        if s >= args.warmup:
            vals.append(v); work += w
    value = float(np.mean(vals))
    cores = blas_threads()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * work / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(cfg, req),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------- GPU bench
def replica_config(base, rank: int):
    """Every rank is an independent replica with its own seeded batch."""
    return small_variant(base, seed=base.seed + 1000 * rank)


def aggregate(dist, t):
    """t = [ms_per_step, attn_ms, e2e_seconds, tokens_per_step, e2e_tokens] of this rank.
    Times are the maximum over ranks, token counts the sum (whole-job throughput)."""
    if dist is not None:
        tmax = t.clone()
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tsum = t.clone()
        dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
    else:
        tmax = tsum = t
    return float(tmax[0]), float(tmax[1]), float(tmax[2]), float(tsum[3]), float(tsum[4])


def run_ours(args, rank, world, local_rank):
    import paper_2609_37532_b200 as P
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    base = CONFIGS[args.workload]
    cfg = replica_config(base, rank)
    if args.layers:
        cfg = small_variant(cfg, layers=args.layers)
    req = make_requests(cfg)
    n_bs, n = req["n_bs"], req["n_live"]
    ws = P.VerifyWorkspace(n_bs, cfg.n_q_heads, cfg.n_kv_heads, device=dev)

    d_n_live = torch.tensor([n], dtype=torch.int32, device=dev)
    d_scores = torch.as_tensor(req["scores"]).to(dev)
    d_draft = torch.as_tensor(req["draft_tokens"]).to(dev)
    d_ctx = torch.as_tensor(req["ctx_len"]).to(dev)
    d_bt = torch.as_tensor(req["block_table"]).to(dev).contiguous()

    def do_alloc():
        P.alloc_verify(ws, d_n_live, d_scores, d_draft, d_ctx, d_bt, req["num_pages"])

    do_alloc()
    torch.cuda.synchronize()
    k = ws.field("k").cpu().numpy().copy()
    offset = ws.field("offset").cpu().numpy().copy()
    assert int(k[:n].sum()) == 8 * n and ws.status() == 0

    layers = []
    for l in range(cfg.layers):
        kc, vc = make_kv_layer(req, l, device=str(dev), poison=False)
        qp = rows_to_packed(make_q_unpacked(req, l, device=str(dev)), k, offset, n, 8 * n_bs)
        layers.append((qp.contiguous(), kc, vc, torch.empty_like(qp)))
    lu = make_logits_unpacked(req, device=str(dev))
    logits = rows_to_packed(lu, k, offset, n, 8 * n_bs).contiguous()
    del lu
    outs = [torch.zeros(n_bs, dtype=torch.int32, device=dev), torch.zeros(n_bs, dtype=torch.int32, device=dev),
            torch.zeros((n_bs, 16), dtype=torch.int32, device=dev), torch.zeros(n_bs, dtype=torch.int32, device=dev)]

    attn = P.verify_attn if args.attn == "tensor" else P.verify_attn_simt

    def do_attn():
        for (q, kc, vc, o) in layers:
            attn(ws, q, kc, vc, d_bt, SCALE, o)

    def do_accept():
        P.accept(ws, logits, cfg.vocab, outs[0], outs[1], outs[2], outs[3], None)

    def step_direct():
        do_alloc(); do_attn(); do_accept()

    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        step_direct()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step_direct()
    torch.cuda.synchronize()
    tokens_per_step = int(outs[3].sum().item())

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    per_layer_b, per_step_b = algorithmic_bytes(cfg, req, k)
    step_bytes = per_layer_b * cfg.layers + per_step_b
    # A step whose inputs fit the 126 MB L2 is timed cold: a buffer larger than the L2 is
    # rewritten before every replay (outside the per-replay events) and the step time is the
    # sum of the per-replay intervals; the back-to-back (warm) figure is reported beside it.
    flush = step_bytes < 4 * L2_BYTES
    flush_buf = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev) if flush else None

    def timed_replays(g, count, cold):
        """Per-replay device times in ms (events on the launching stream)."""
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(2 * count)]
        for s_ in range(count):
            if cold:
                flush_buf.fill_(s_ & 1)
            evs[2 * s_].record(stream)
            g.replay()
            evs[2 * s_ + 1].record(stream)
        barrier()
        return np.array([evs[2 * s_].elapsed_time(evs[2 * s_ + 1]) for s_ in range(count)])

    def time_captured(fn, inner=8, reps=None):
        """Per-call device time in ms of fn(): `inner` calls captured as one graph (what a step
        does with every call of this library), median over the replays."""
        fn()
        barrier()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(inner):
                fn()
        g.replay()
        barrier()
        reps = reps or max(5, min(args.steps, 20))
        return float(np.median(timed_replays(g, reps, cold=False))) / inner

    sampler = ClockSampler(local_rank)
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            graph.replay()
        barrier()
        if rank == 0:
            sampler.start()
        # ---- timed region 1: K replays of the captured step (headline) ----
        barrier()
        if flush:
            per_replay = timed_replays(graph, args.steps, cold=True)
            ms_total = float(per_replay.sum())
            warm_ms = float(np.median(timed_replays(graph, args.steps, cold=False)))
        else:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            e0.record(stream)
            marks[0].record(stream)
            for s_ in range(args.steps):
                graph.replay()
                marks[s_ + 1].record(stream)
            e1.record(stream)
            barrier()
            ms_total = e0.elapsed_time(e1)
            per_replay = np.array([marks[s_].elapsed_time(marks[s_ + 1]) for s_ in range(args.steps)])
            warm_ms = None

        # ---- timed region 2: the dominant kernel alone, for its roofline: the L
        # attention launches of a step captured as their own graph (same launch
        # configuration as in the step), K replays, CUDA events around each ----
        g_attn = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_attn, stream=stream):
            do_attn()
        g_attn.replay()
        barrier()
        _per = timed_replays(g_attn, args.steps, cold=flush) / max(1, cfg.layers)
        attn_ms = float(np.mean(_per))
        attn_med_ms, attn_min_ms = float(np.median(_per)), float(_per.min())
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # argmax + acceptance alone: copies of the logits taken in turn (four sets, 4 x the size of L2 at
        # the full step), so that no call finds its rows in L2; the sets hold the same values
        accept_bytes = 8 * n * cfg.vocab * 4
        logit_sets = [logits] + [logits.clone() for _ in range(3 if 4 * accept_bytes < (8 << 30) else 0)]
        turn = [0]

        def accept_next():
            lg = logit_sets[turn[0] % len(logit_sets)]
            turn[0] += 1
            P.accept(ws, lg, cfg.vocab, outs[0], outs[1], outs[2], outs[3], None)
        accept_ms = time_captured(accept_next)
        del logit_sets[1:]
        # the sampling verifier (temperature 1) on the same logits, for its own figure
        u_acc = torch.rand(8 * n_bs, device=dev)
        u_drw = torch.rand(n_bs, device=dev)
        so = [torch.zeros_like(outs[0]), torch.zeros_like(outs[1]), torch.zeros_like(outs[2]), torch.zeros_like(outs[3])]
        sampling_ms = time_captured(
            lambda: P.accept_sampling(ws, logits, cfg.vocab, 1.0, u_acc, u_drw, so[0], so[1], so[2], so[3]))

        # the fused LM head + argmax + acceptance (one launch) on seeded hidden states
        lm = None
        if args.lm_hidden > 0:
            w_lm, h_un = make_lm_head_unpacked(req, args.lm_hidden, device=str(dev))
            h_lm = rows_to_packed(h_un, k, offset, n, 8 * n_bs)
            del h_un
            lo = [torch.zeros_like(x) for x in outs[:4]]
            lm_ms = time_captured(lambda: P.lm_head_accept(ws, h_lm, w_lm, lo[0], lo[1], lo[2], lo[3]), inner=4)
            # context: the library GEMM that would only produce the logits (bf16 out)
            for _ in range(2):
                lg = torch.matmul(h_lm, w_lm.t())
            ea.record(stream)
            for _ in range(args.steps):
                lg = torch.matmul(h_lm, w_lm.t())
            eb.record(stream)
            barrier()
            gemm_ms = ea.elapsed_time(eb) / args.steps
            lm_bytes = w_lm.numel() * 2 + h_lm.numel() * 2
            lm_flops = 2.0 * 8 * n * cfg.vocab * args.lm_hidden
            lm = {"us": lm_ms * 1e3, "hidden": args.lm_hidden, "bytes": lm_bytes,
                  "gbs": lm_bytes / (lm_ms * 1e-3) / 1e9, "tflops": lm_flops / (lm_ms * 1e-3) / 1e12,
                  "library_gemm_logits_only_us": gemm_ms * 1e3,
                  # both roofs lie close together at 256 rows: report the fraction of each
                  "frac_of_hbm_peak": lm_bytes / (lm_ms * 1e-3) / 1e9 / measured_peak()[0],
                  "frac_of_bf16_peak": lm_flops / (lm_ms * 1e-3) / 1e12 / measured_bf16_peak()}
            del w_lm, h_lm, lg

        # the predictor front end (two launches) on seeded drafter outputs
        pred = None
        if args.pred_hidden > 0:
            pin = make_predictor_inputs(req, args.pred_hidden, device=str(dev))
            pl_out = torch.zeros((n_bs, 15), dtype=torch.float32, device=dev)

            def do_pred():
                P.predict_scores(ws, d_n_live, pin["draft_logits"], cfg.vocab, pin["draft_hidden"], pin["p_hidden"],
                                 pin["p_logit"], pin["w1"], pin["b1"], pin["w2"], pin["b2"], pl_out)
            pred_ms = time_captured(do_pred, inner=4)
            pred_bytes = 15 * n * cfg.vocab * 4 + 32 * cfg.vocab * 2 + 15 * n * args.pred_hidden * 2
            pred = {"us": pred_ms * 1e3, "hidden": args.pred_hidden, "bytes": pred_bytes,
                    "gbs": pred_bytes / (pred_ms * 1e-3) / 1e9,
                    "frac_of_hbm_peak": pred_bytes / (pred_ms * 1e-3) / 1e9 / measured_peak()[0]}
            del pin

        # ---- sustained legs: the same two graphs replayed for seconds, so that the clock has
        # settled under the power cap; per-replay times over the last two thirds of the run
        sustained = None
        if args.sustain_s > 0 and not flush:
            def sustained_leg(g, seconds, per_replay_ms):
                smp = ClockSampler(local_rank)
                count = max(20, int(seconds * 1e3 / per_replay_ms))
                evs = [torch.cuda.Event(enable_timing=True) for _ in range(count + 1)]
                barrier()
                smp.start()
                t_wall = time.perf_counter()
                evs[0].record(stream)
                for s_ in range(count):
                    g.replay()
                    evs[s_ + 1].record(stream)
                barrier()
                wall = time.perf_counter() - t_wall
                clk = smp.stop()
                per = np.array([evs[s_].elapsed_time(evs[s_ + 1]) for s_ in range(count)])
                tail = per[count // 3:]
                return {"replays": count, "wall_s": wall, "median_ms": float(np.median(tail)),
                        "min_ms": float(tail.min()), "first_ms": float(np.median(per[:5])),
                        "sm_mhz": clk.get("sm_mhz"), "reasons": clk.get("reasons")}
            st_step = sustained_leg(graph, args.sustain_s, ms_total / args.steps)
            st_attn = sustained_leg(g_attn, args.sustain_s * 2.0 / 3.0, attn_ms * cfg.layers)
            sustained = {"step": st_step, "attn": st_attn}

        # ---- the whole decision chain as one captured graph (Algorithm 2: features ->
        # DVL, then target -> accept -> output): predictor front end -> allocation from its
        # logits -> attention x L -> fused LM head + acceptance, on seeded drafter outputs
        chain = None
        if args.chain and args.lm_hidden > 0 and args.pred_hidden > 0 and args.attn == "tensor":
            pin = make_predictor_inputs(req, args.pred_hidden, device=str(dev))
            w_lm, h_un = make_lm_head_unpacked(req, args.lm_hidden, device=str(dev))
            h_lm = rows_to_packed(h_un, k, offset, n, 8 * n_bs)
            del h_un
            pl_out = torch.zeros((n_bs, 15), dtype=torch.float32, device=dev)
            co = [torch.zeros_like(x) for x in outs[:4]]

            def chain_step():
                P.predict_scores(ws, d_n_live, pin["draft_logits"], cfg.vocab, pin["draft_hidden"], pin["p_hidden"],
                                 pin["p_logit"], pin["w1"], pin["b1"], pin["w2"], pin["b2"], pl_out)
                P.alloc_verify(ws, d_n_live, pl_out, d_draft, d_ctx, d_bt, req["num_pages"], scores_are_logits=True)
                do_attn()
                P.lm_head_accept(ws, h_lm, w_lm, co[0], co[1], co[2], co[3])
            chain_step()
            barrier()
            g_chain = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_chain, stream=stream):
                chain_step()
            for _ in range(3):
                g_chain.replay()
            barrier()
            ch = timed_replays(g_chain, max(5, min(args.steps, 20)), cold=False)
            k_chain = ws.field("k").cpu().numpy().copy()
            kv_len = req["ctx_len"][:n].astype(np.int64) + k_chain[:n].astype(np.int64)
            chain_bytes = (int(kv_len.sum()) * cfg.n_kv_heads * 128 * 2 * 2 + int(((kv_len + 15) // 16).sum()) * 4 +
                           2 * 8 * n * cfg.n_q_heads * 128 * 2) * cfg.layers
            chain_bytes += 15 * n * cfg.vocab * 4 + 32 * cfg.vocab * 2 + 15 * n * args.pred_hidden * 2     # drafter outputs
            chain_bytes += w_lm.numel() * 2 + h_lm.numel() * 2                                              # LM head
            ch_ms = float(np.median(ch))
            chain = {"graph": "predict_scores -> alloc_verify (logits) -> verify_attn x %d -> lm_head_accept" % cfg.layers,
                     "ms_per_step": ch_ms, "min_ms": float(ch.min()), "bytes": int(chain_bytes),
                     "gbs": chain_bytes / (ch_ms * 1e-3) / 1e9,
                     "frac_of_hbm_peak": chain_bytes / (ch_ms * 1e-3) / 1e9 / measured_peak()[0],
                     "verified_tokens_per_step": int(co[3].sum().item()),
                     "gpu_launches_per_step": P.lib.dscale_launches_per_call(7) + P.lib.dscale_launches_per_call(0) +
                                              cfg.layers * P.lib.dscale_launches_per_call(1) + P.lib.dscale_launches_per_call(6)}
            del pin, w_lm, h_lm, g_chain
            do_alloc()                          # the workspace back to the canonical allocation
            barrier()

        # ---- timed region 3: end to end through the host-buffer C ABI call ----
        hs = P.HostStep(ws, req["max_pages"], req["num_pages"], layers, logits, cfg.vocab, SCALE)
        hs.h_n_live[0] = n
        hs.h_scores.copy_(torch.as_tensor(req["scores"]))
        hs.h_draft.copy_(torch.as_tensor(req["draft_tokens"]))
        hs.h_ctx_len.copy_(torch.as_tensor(req["ctx_len"]))
        hs.h_block_table.copy_(torch.as_tensor(req["block_table"]))
        for _ in range(max(1, args.warmup)):
            hs.run(graph=True); stream.synchronize()
        barrier()
        t0 = time.perf_counter()
        e2e_tokens = 0
        for _ in range(args.steps):
            hs.run(graph=True)
            stream.synchronize()                      # the caller reads the outputs every step
            e2e_tokens += int(hs.h_out_len.sum())
        e2e_s = time.perf_counter() - t0
    clocks = sampler.stop() if rank == 0 else None
    assert ws.status() == 0, f"device status {ws.status()}"

    ms_step = ms_total / args.steps
    t = torch.tensor([ms_step, attn_ms, e2e_s, float(tokens_per_step), float(e2e_tokens)],
                     dtype=torch.float64, device=dev)
    ms_step, attn_ms, e2e_s, tokens_all, e2e_tokens_all = aggregate(dist, t)
    value = tokens_all / (ms_step * 1e-3)
    e2e_value = e2e_tokens_all / e2e_s

    if rank == 0:
        peak, peak_kind = measured_peak()
        achieved = per_layer_b / (attn_ms * 1e-3) / 1e9
        step_gbs = (per_layer_b * cfg.layers + per_step_b) / (ms_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(cfg, req, args.attn),
            "verified_tokens_per_step": tokens_per_step,
            "step_ms": {"mean": ms_step, "median": float(np.median(per_replay)), "min": float(per_replay.min()),
                        "warm_median": warm_ms},
            "sustained": sustained,
            "decision_chain": chain,
            "packed_rows_per_s": 8 * n * world / (ms_step * 1e-3),
            "step_gbs": step_gbs, "step_frac_of_peak": step_gbs / peak,
            "step_frac_of_8tbs": step_gbs / 8000.0,
            "roofline": {"bound": "hbm", "kernel": "attn_tc_kernel" if args.attn == "tensor" else "attn_simt_kernel",
                         "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                         "frac": achieved / peak, "frac_of_8tbs": achieved / 8000.0,
                         "bytes_per_launch": per_layer_b, "us_per_launch": attn_ms * 1e3,
                         "us_per_launch_median": attn_med_ms * 1e3, "us_per_launch_min": attn_min_ms * 1e3,
                         "frac_sustained": (per_layer_b / (sustained["attn"]["median_ms"] / cfg.layers * 1e-3) / 1e9 / peak)
                                           if sustained else None,
                         "us_per_launch_sustained": (sustained["attn"]["median_ms"] / cfg.layers * 1e3) if sustained else None,
                         "traffic": recorded_traffic(cfg.name)},
            "accept_us": accept_ms * 1e3, "accept_gbs": accept_bytes / (accept_ms * 1e-3) / 1e9,
            "accept_frac_of_hbm_peak": accept_bytes / (accept_ms * 1e-3) / 1e9 / measured_peak()[0],
            "accept_sampling_us": sampling_ms * 1e3,
            "lm_head_accept": lm, "predict_scores": pred,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": hs.h2d_bytes,
                    "d2h_bytes_per_step": hs.d2h_bytes, "ms_per_step": 1e3 * e2e_s / args.steps,
                    "api": "dscale_verify_step_host_graph (pinned host inputs/outputs, KV/Q/logits resident)"},
            "gpu_launches": args.steps * (P.lib.dscale_launches_per_call(0) +
                                          cfg.layers * P.lib.dscale_launches_per_call(1 if args.attn == "tensor" else 3) +
                                          P.lib.dscale_launches_per_call(2)),
            "clocks": clocks,
        }
        if world == 1 and not args.no_padded:
            # the in-repo comparison: unpacked W = 16, one 128-row tile per (request, q-head)
            with torch.cuda.stream(stream):
                qus = [make_q_unpacked(req, l, device=str(dev)) for l in range(cfg.layers)]
                ous = [torch.empty_like(q) for q in qus]

                def do_padded():
                    for l, (q, kc, vc, o) in enumerate(layers):
                        P.verify_attn_padded(ws, qus[l], kc, vc, d_bt, d_ctx, SCALE, ous[l])
                do_padded()
                pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                n_rep = max(1, min(args.steps, 5))
                pa.record(stream)
                for _ in range(n_rep):
                    do_padded()
                pb.record(stream)
                torch.cuda.synchronize()
                pad_us = 1e3 * pa.elapsed_time(pb) / n_rep / max(1, cfg.layers)
            line["padded_baseline"] = {
                "what": "unpacked W=16 verify attention, 128-row tile per (request, q-head), 16N rows",
                "attn_us_per_launch": pad_us, "packed_attn_us_per_launch": attn_ms * 1e3,
                "attn_speedup_packed_vs_padded": pad_us / (attn_ms * 1e3)}
            del qus, ous
        if world == 1 and not args.no_cpu_baseline:
            n_l = min(cfg.layers, args.cpu_layers)
            kvs = [(layers[l][1].cpu(), layers[l][2].cpu()) for l in range(n_l)]
            qus = [make_q_unpacked(req, l, device=str(dev)).cpu() for l in range(n_l)]
            lu_cpu = make_logits_unpacked(req, device=str(dev)).cpu()
            v, work, desc = oracle_step_sample(cfg, req, kvs, qus, lu_cpu)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": desc, "cpu_seconds": work}
            try:                                 # the same oracle on one thread, on a smaller sample
                from threadpoolctl import threadpool_limits
                n_1 = max(1, min(2, n_l))
                with threadpool_limits(limits=1):
                    v1, work1, desc1 = oracle_step_sample(cfg, req, kvs[:n_1], qus[:n_1], lu_cpu)
                line["cpu_baseline"]["single_thread"] = {"value": v1, "unit": UNIT, "cores": 1, "sample": desc1,
                                                         "cpu_seconds": work1}
            except Exception as e:               # threadpoolctl missing: say so, keep the threaded figure
                line["cpu_baseline"]["single_thread"] = {"unavailable": str(e)}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3_8b_step", choices=list(CONFIGS))
    ap.add_argument("--attn", default="tensor", choices=["tensor", "simt"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling)")
    ap.add_argument("--lm-hidden", type=int, default=4096,
                    help="hidden size of the fused LM-head figure (0 skips it)")
    ap.add_argument("--pred-hidden", type=int, default=4096,
                    help="drafter hidden size of the predictor front-end figure (0 skips it)")
    ap.add_argument("--sustain-s", type=float, default=3.0,
                    help="seconds of back-to-back replays for the sustained legs (0 skips them)")
    ap.add_argument("--no-chain", dest="chain", action="store_false",
                    help="skip the full-size decision-chain graph (predictor -> allocation -> attention -> LM head)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-padded", action="store_true", help="skip the padded comparison kernel")
    ap.add_argument("--cpu-layers", type=int, default=0,
                    help="layers of attention the CPU oracle is timed on (its time is scaled to all "
                         "layers); default 12 for the cpu_baseline leg, 2 per step for --impl reference")
    args = ap.parse_args()
    if args.cpu_layers <= 0:
        args.cpu_layers = 18 if args.impl == "ours" else 2
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local_rank = int(os.environ.get("LOCAL_RANK", 0))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
