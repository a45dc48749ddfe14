#!/usr/bin/env python
"""Throughput of one n-wise training step (tokens/s) on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--n 2] [--impl reference]
                    [--head-mode stored|recompute] [--placement replicas|pipeline]

A step is the whole hot path on one batch: il_set_batch, K x (il_forward_component, il_aux_head_loss),
il_backward_nwise and, where the configuration says so, il_adamw_step.  The default workload is the
GPT-2-medium-shaped configuration (24 layers in 8 components, d 1024, seq 1024, batch 8, vocab 50257,
n = 2, AdamW).  With N > 1 (launched under torch.distributed.run) every rank runs an independent
replica of the same step on its own GPU: the path has no exchange step, so there is no collective on
the data path and the scaling is weak.  Rank 0 prints one JSON line.

`--placement pipeline` times the paper's own placement instead (Sec. 3: one module per accelerator): one process
drives all N GPUs, component k lives on GPU k*N//K, boundary activations and passed-down gradients are copied into
buffers the receiving GPU owns.  Under torch.distributed.run rank 0 does this alone and the other ranks exit.  The
line then also carries the time per batch of the paper's model (Sec. 3.1) with its slot cost fitted to the measured
1-wise step of the same placement.

`--impl reference` times the fp64 CPU oracle, as it stands, on the host cores on a bounded sample of
the same workload (one sequence of the batch).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402


# DRAM bytes per algorithmic flop of the GEMM kernel, from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum over all 270 GEMM launches of a cfg4-2x1 run, whose launch shapes are cfg4's).
# Traffic grows with the flops of a launch at fixed shapes, so the
# per-launch figure of another step mix is this ratio times that mix's flops per launch.  Set to None whenever
# gemm.cu changes after the capture.
GEMM_DRAM_BYTES_PER_FLOP = 1.2558e-3


def model_flops_per_token(w: wl.Workload, n: int) -> float:
    """Algorithmic flops per token of one n-wise step: every contraction the method defines, counted once
    (forward, one wgrad per matrix, one dgrad per distinct gradient stream); recomputation is not counted."""
    gemm = 2.0 * (3 * w.d * w.d + w.d * w.d + 2 * w.d * w.F)          # per layer, forward
    att_f = 2.0 * w.T * w.d                                            # causal QK^T + PV
    att_b = 4.0 * w.T * w.d
    total = 0.0
    for k in range(w.K):
        heads = [h for h in range(w.K) if max(h - n + 1, 0) <= k <= h]
        if w.rule == "sum":
            s_k = len({max(h - n + 1, 0) for h in heads})
        else:
            # weighted rules: one stream for the weighted combination that drives the parameter gradients plus
            # one per head that continues below the component (the two coincide when a single head is involved)
            below = [h for h in heads if k > 0 and h < k + n - 1]
            s_k = 1 + len(below) - (1 if len(heads) == 1 and below else 0)
        total += w.Lc * (gemm + att_f) + w.Lc * gemm + s_k * w.Lc * (gemm + att_b)
    total += w.K * 6.0 * w.d * w.V
    # blocks inside the auxiliary heads: forward, wgrad and one dgrad each
    total += w.K * w.Lh * ((gemm + att_f) + gemm + (gemm + att_b))
    return total


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(w: wl.Workload, n: int, steps: int, warmup: int, params=None, budget_s: float = 25.0):
    """Time the oracle (fp64, numpy), as it stands, on a bounded sample of the workload: the first
    positions of one sequence of the batch, the sample length chosen so that the whole call takes about
    `budget_s` seconds of host time.  Returns (tokens/s, seconds per step, info)."""
    from oracle import il_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    est_per_token = model_flops_per_token(w, n) / 45e9          # observed oracle rate on 8 cores, rough
    ts = int(budget_s / max(steps + warmup, 1) / est_per_token) // 32 * 32
    ts = max(32, min(ts, w.T))
    ws = w.with_(B=1, T=ts)
    P = params if params is not None else wl.draw_params(w)
    tok, tgt = wl.draw_tokens(w)
    tok, tgt = np.ascontiguousarray(tok[:1, :ts]), np.ascontiguousarray(tgt[:1, :ts])
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.nwise_gradients(P, tok, tgt, ws.K, ws.Lc, ws.H, n, rule=ws.rule, head_layers=ws.Lh)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times))
    info = {"value": ws.ntok / sec, "unit": "tokens/s", "cores": int(cores), "kind": "oracle",
            "sample": f"{len(times)} oracle step(s) (forward, K heads, per-head n-wise backward; no optimiser) on the "
                      f"first {ts} positions of 1 of {w.B} sequences of {w.name} (full model, n={n}); "
                      f"{sec:.2f} s per step"}
    # The short sample is dominated by costs that do not grow with the tokens (every weight matrix is widened to
    # fp64 and read once per step whatever the batch), so two more figures are given: the sample scaled to the full
    # step by the ratio of algorithmic flops, and the oracle's own time for the full-size step where the run that
    # wrote the stored expected values recorded it.
    full_flops = model_flops_per_token(w, n) * w.ntok
    sample_flops = model_flops_per_token(ws, n) * ws.ntok
    sec_full = sec * full_flops / sample_flops
    info["live_extrapolation"] = {"value": w.ntok / sec_full, "unit": "tokens/s", "seconds_per_full_step": sec_full,
                                  "how": "live sample time x (algorithmic flops of the full step / of the sample)"}
    gold = os.path.join(ROOT, "tests", "golden", f"{w.name}_n{n}.json")
    info["cached_full_run"] = None
    if os.path.exists(gold):
        try:
            g = json.load(open(gold))
            if g.get("oracle_seconds"):
                info["cached_full_run"] = {"value": w.ntok / float(g["oracle_seconds"]), "unit": "tokens/s",
                                           "seconds_per_full_step": float(g["oracle_seconds"]),
                                           "cores": g.get("oracle_cores", 8),
                                           "how": "wall time of the oracle's full-size step (with the summaries it "
                                                  "stores) on the machine that wrote tests/golden"}
        except Exception:
            pass
    return ws.ntok / sec, sec, info


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the whole job = the slowest replica's (the replicas never exchange data)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_rank_step: int, steps: int, world: int, ms: float) -> float:
    """Whole-job throughput of `world` independent replicas over `steps` steps lasting `ms` (max over ranks)."""
    return tokens_per_rank_step * steps * max(world, 1) / (ms * 1e-3)


def bench_pipeline(args, w, n, metric, cfg_desc):
    """One process, N GPUs, component k on GPU k*N//K (Sec. 3: one module per accelerator; several modules on one
    accelerator are merged).  Times the requested n and n = 1 and sets them beside the paper's time-per-batch
    model T(A, 1, N) = 2 N c (Sec. 3.1) with the slot cost c taken from the measured 1-wise step."""
    import torch
    from paper_2010_04116_b200 import Model, time_per_batch

    ngpu = max(1, min(args.gpus, torch.cuda.device_count(), w.K))
    devices = [k * ngpu // w.K for k in range(w.K)]
    use_adamw = bool(w.adamw and not args.no_adamw)
    hp = dict(lr=1e-4, beta1=0.9, beta2=0.98, eps=1e-9, weight_decay=w.weight_decay) if use_adamw else None
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B // w.M, w.T, device=0, head_layers=w.Lh, head_mode=args.head_mode,
              placement="pipeline", devices=devices, attn_bwd=args.attn_bwd)
    if w.rule != "sum":
        m.set_rule(w.rule)
    if w.M > 1:
        m.set_micro_batches(w.M)
    params = wl.draw_params(w)
    m.set_params(params)
    dev0 = torch.device("cuda", 0)
    nb = 4
    batches = [tuple(torch.tensor(x, device=dev0) for x in wl.draw_tokens(w, step=s)) for s in range(nb)]

    def run(count):
        for i in range(count):
            tok, tgt = batches[i % nb]
            if w.M > 1:
                if hp is None:
                    m.set_micro_batches(w.M)
                m.train_minibatch(tok, tgt, w.M, adamw=hp)
            else:
                m.train_step(tok, tgt, adamw=hp)

    def timed(count):
        m.sync()
        s0 = m.streams[0]
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.device(0):
            start.record(s0)
            run(count)
            for s in m.streams[1:]:
                s0.wait_stream(s)
            end.record(s0)
        m.sync()
        return start.elapsed_time(end)

    results = {}
    sampler = ClockSampler(0)
    for nn in sorted({1, n}):
        m.set_n(nn)
        run(max(args.warmup, 3))
        if nn == n:
            sampler.start()
        results[nn] = timed(args.steps) / args.steps
    clocks = sampler.stop()
    launches_per_step = None
    l0 = m.stats()[1]
    run(1)
    m.sync()
    launches_per_step = m.stats()[1] - l0
    transfers = m.last_transfers()
    c = results[1] / 2.0
    model_ms = time_per_batch(w.K, 1, n, c, 0.0)
    flops_tok = model_flops_per_token(w, n)
    value = w.ntok / (results[n] * 1e-3)
    out = {"metric": metric, "value": value, "unit": "tokens/s", "n_gpus": ngpu, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": results[n], "higher_is_better": True, "scaling": "strong",
           "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": dict(cfg_desc, parallelism=f"pipeline placement: {w.K} components on {ngpu} GPU(s), map {devices}",
                          global_batch=w.B),
           "clocks": clocks, "gpu_launches": int(launches_per_step * args.steps),
           "placement": {"devices": devices,
                         "copies_per_step": {"forward": sum(1 for t in transfers if t[0] == 0),
                                             "backward": sum(1 for t in transfers if t[0] == 1)},
                         "bytes_per_copy": int(w.ntok // w.M * w.d * 4),
                         "ms_per_step_1wise": results[1]},
           "timing_model": {"A": w.K, "M": 1, "N": n, "slot_cost_ms": c, "time_per_batch_ms": model_ms,
                            "measured_ms": results[n],
                            "note": ("Sec. 3.1: T = 2 N c for M = 1, c fitted as half the measured 1-wise step of this "
                                     "placement; the model describes one accelerator per module, so it applies when "
                                     f"n_gpus = {w.K}" + ("" if ngpu == w.K else f" (this run: {ngpu})"))},
           "model_flops": {"per_token_mflop": flops_tok / 1e6, "tflops_whole_job": value * flops_tok / 1e12},
           "e2e": None, "roofline": None, "cpu_baseline": None}
    m.close()
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="cfg4")
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-adamw", action="store_true")
    ap.add_argument("--head-mode", default="stored", choices=["stored", "recompute"])
    ap.add_argument("--placement", default="replicas", choices=["replicas", "pipeline"])
    ap.add_argument("--attn-bwd", default="one_sweep", choices=["one_sweep", "two_kernels"])
    ap.add_argument("--no-head-mode-comparison", action="store_true")
    args = ap.parse_args()

    w = wl.CONFIGS[args.config]
    n = args.n if args.n is not None else w.n
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    metric = "training tokens/s per n-wise step"
    extra = (f", {w.Lh} blocks per auxiliary head, rule={w.rule}, {w.M} micro-batches per update"
             if (w.Lh or w.M > 1 or w.rule != "sum") else "")
    cfg_desc = {"workload": f"{w.name}: {w.K}x{w.Lc} layers, d={w.d}, H={w.H}, F={w.F}, T={w.T}, B={w.B}, V={w.V}, "
                            f"n={n}, adamw={bool(w.adamw and not args.no_adamw)}{extra}, head_mode={args.head_mode}, attn_bwd={args.attn_bwd}",
                "global_batch": w.B * max(world, 1), "seq_len": w.T, "parallelism": f"replicas x{max(world, 1)}",
                "l2": "inputs larger than L2 (each step streams several GB of weights and activations)"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps, warm = max(1, args.steps), max(0, args.warmup)
        val, sec, info = oracle_sample(w, n, steps, warm, budget_s=150.0)
        info = dict(info, value=val)
        print(json.dumps({"impl": "reference", "metric": metric, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
                          "steps": steps, "warmup": warm, "ms_per_step": sec * 1e3, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                          "config": cfg_desc, "cpu_baseline": info,
                          "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    from paper_2010_04116_b200 import Model

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    if args.placement == "pipeline":
        if rank == 0:
            bench_pipeline(args, w, n, metric, cfg_desc)
        return
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    use_adamw = bool(w.adamw and not args.no_adamw)
    hp = dict(lr=1e-4, beta1=0.9, beta2=0.98, eps=1e-9, weight_decay=w.weight_decay) if use_adamw else None
    m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B // w.M, w.T, device=local_rank, head_layers=w.Lh,
              head_mode=args.head_mode, attn_bwd=args.attn_bwd)
    if w.rule != "sum":
        m.set_rule(w.rule)
    if w.M > 1:
        m.set_micro_batches(w.M)
    # parameters drawn on the host by the seeded generator, copied once
    params = wl.draw_params(w)
    m.set_params(params)
    nb = 4
    batches = [wl.draw_tokens(w, step=s) for s in range(nb)]
    dev = torch.device("cuda", local_rank)
    dev_batches = [(torch.tensor(a, device=dev), torch.tensor(b, device=dev)) for a, b in batches]
    pin_batches = [(torch.tensor(a).pin_memory(), torch.tensor(b).pin_memory()) for a, b in batches]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    s0 = m.streams[0]

    def run_steps(count, e2e):
        for i in range(count):
            tok, tgt = (pin_batches if e2e else dev_batches)[i % nb]
            if w.M > 1:
                if hp is None:
                    m.set_micro_batches(w.M)     # no update follows: start the next accumulation explicitly
                m.train_minibatch(tok, tgt, w.M, adamw=hp)
            else:
                m.train_step(tok, tgt, adamw=hp)
            if e2e:
                m.get_losses()          # device -> host read of the step's result (waits for the heads)

    def timed(count, e2e):
        barrier()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(s0)
        run_steps(count, e2e)
        for s in m.streams[1:]:
            s0.wait_stream(s)
        end.record(s0)
        barrier()
        m.sync()
        return max_over_ranks(start.elapsed_time(end), dist, dev)

    run_steps(args.warmup, False)
    m.sync()
    l0 = m.stats()[1]
    sampler = ClockSampler(local_rank)
    sampler.start()
    ms = timed(args.steps, False)
    clocks = sampler.stop()
    launches = m.stats()[1] - l0
    # Two more steps with every GEMM alone on the GPU (a pair of CUDA events around each, all other streams held
    # back meanwhile) give the kernel's own durations at the step's launch shapes, straight after the timed steps.
    m.profile(2)
    run_steps(2, False)
    m.sync()
    x_ms, x_launches, x_flops = m.profile_read()
    m.profile(False)
    # The K steps once more with a pair of CUDA events around every GEMM launch (on the launch's own stream): the
    # GEMM kernel's durations inside a running step, where the component streams share the GPU and the intervals
    # include waiting for SMs.  The events cost time of their own (two records per GEMM,
    # and a kernel between events cannot set itself up while its predecessor drains), so these steps are not the
    # ones the headline value is taken from; their step time is reported beside the figure.
    m.profile(True)
    ms_events = timed(args.steps, False)
    gemm_ms, gemm_launches, gemm_flops = m.profile_read()
    m.profile(False)
    losses = m.get_losses() if not use_adamw else None
    # end to end: pinned host tokens copied in, losses read back, every step
    run_steps(1, True)
    ms_e2e = timed(args.steps, True)

    value = job_tokens_per_s(w.ntok, args.steps, world, ms)
    e2e = job_tokens_per_s(w.ntok, args.steps, world, ms_e2e)
    flops_tok = model_flops_per_token(w, n)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak_sus = float(peaks.get("bf16_tflops_sustained", 1400.0))
    peak_burst = float(peaks.get("bf16_tflops", 1590.0))
    peak_src = "measured (MEASURED_PEAKS.json, sustained bf16 matmul)" if peaks else "fallback (1.4 PFLOP/s sustained)"
    achieved_shared = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    achieved = x_flops / (x_ms * 1e-3) / 1e12 if x_ms > 0 else 0.0
    per_gpu_tf = value / max(world, 1) * flops_tok / 1e12
    out = {
        "metric": metric, "value": value, "unit": "tokens/s", "n_gpus": max(world, 1), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg_desc, "clocks": clocks,
        "e2e": {"value": e2e, "unit": "tokens/s", "h2d_bytes_per_step": int(2 * w.ntok * 4),
                "d2h_bytes_per_step": int(4 * w.K), "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "gemm_tcgen05_kernel (all layouts and epilogues)",
                     "achieved": achieved, "peak": peak_sus, "unit": "TFLOP/s", "frac": achieved / peak_sus,
                     "peak_source": peak_src, "launches": int(x_launches), "avg_launch_ms": x_ms / max(x_launches, 1),
                     "how": "sum of 2MNK over every GEMM launch of two steps / sum of their CUDA-event durations with "
                            "each GEMM alone on the GPU",
                     "timed_region": {"achieved": achieved_shared, "launches": int(gemm_launches),
                                      "gemm_share_of_step": gemm_ms / ms_events if ms_events > 0 else None,
                                      "ms_per_step_with_events": ms_events / args.steps,
                                      "note": "the K timed steps repeated with a pair of events around every GEMM on its "
                                              "launch stream; intervals overlap across the component streams and "
                                              "include waiting for SMs; the events themselves lengthen the step, so "
                                              "the headline value comes from the K steps without them"},
                     "traffic": (GEMM_DRAM_BYTES_PER_FLOP * x_flops / max(x_launches, 1)
                                 if GEMM_DRAM_BYTES_PER_FLOP and w.name.startswith("cfg4") else None),
                     "traffic_note": "DRAM bytes per launch = measured bytes/flop of the same launch shapes (ncu, "
                                     "cfg4-2x1) x this run's flops per launch; algorithmic operand+output bytes are "
                                     "of the same size (no re-reads)"},
        "model_flops": {"per_token_mflop": flops_tok / 1e6, "step_tflop": flops_tok * w.ntok / 1e12,
                        "tflops_per_gpu": per_gpu_tf, "frac_of_burst_peak": per_gpu_tf / peak_burst,
                        "frac_of_sustained_peak": per_gpu_tf / peak_sus, "burst_peak": peak_burst},
    }
    if losses is not None:
        out["last_losses"] = [float(x) for x in losses]
    # Per-phase times (a diagnostic beside the step time, not part of it): three more steps with a device
    # synchronisation between the phases, so nothing of one phase overlaps the next; host clock around the syncs.
    if w.M == 1:
        ph = np.zeros(3)
        for i in range(3):
            tok, tgt = dev_batches[i % nb]
            m.sync()
            t0 = time.perf_counter()
            m.set_batch(tok, tgt)
            for k in range(w.K):
                m.forward_component(k)
                m.aux_head_loss(k)
            m.sync()
            t1 = time.perf_counter()
            m.backward_nwise()
            m.sync()
            t2 = time.perf_counter()
            if hp is not None:
                m.adamw_step(**hp)
                m.sync()
            t3 = time.perf_counter()
            ph += np.array([t1 - t0, t2 - t1, t3 - t2]) * 1e3 / 3
        out["phases_ms"] = {"forward_and_head_losses": float(ph[0]), "backward_nwise": float(ph[1]), "adamw": float(ph[2]),
                            "note": "each phase alone on the GPU (synchronised between phases); in the timed step they overlap"}
    dev_bytes = m.stats()[0]
    out["head_mode"] = {"mode": args.head_mode, "ms_per_step": ms / args.steps, "device_bytes": int(dev_bytes)}
    m.close()
    if world == 1 and not args.no_head_mode_comparison:
        # the other head mode on the same workload: step time and device memory side by side
        other = "recompute" if args.head_mode == "stored" else "stored"
        torch.cuda.empty_cache()
        m = Model(w.K, w.Lc, w.d, w.H, w.F, w.V, n, w.B // w.M, w.T, device=local_rank, head_layers=w.Lh, head_mode=other,
                  attn_bwd=args.attn_bwd)
        if w.rule != "sum":
            m.set_rule(w.rule)
        if w.M > 1:
            m.set_micro_batches(w.M)
        m.set_params(params)
        s0 = m.streams[0]
        run_steps(max(args.warmup, 3), False)
        m.sync()
        ms_other = timed(args.steps, False)
        out["head_mode"]["other"] = {"mode": other, "ms_per_step": ms_other / args.steps,
                                     "device_bytes": int(m.stats()[0])}
        m.close()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        _, _, info = oracle_sample(w, n, 1, 0, params=params)
        out["cpu_baseline"] = info
    elif rank == 0:
        out["cpu_baseline"] = None
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
