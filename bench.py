#!/usr/bin/env python
"""Benchmark of the FlowCache hot path on B200: one "step" = decide -> chunk-causal attention ->
score -> top-B select -> gather-compact over one batch of synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the attention work (algorithmic FLOPs of the active
chunks' visible prefixes) divided by the time of the WHOLE step, inputs resident in HBM; `e2e`
is the same with host buffers and the host<->device copies inside the timed region; `roofline`
describes the dominant kernel (attention, tensor-bound) and `roofline_compact` the K/V gather
(HBM-bound); `cpu_baseline` is the CPU oracle timed on a bounded sample of the same workload.
With --impl reference the oracle itself is the timed program (host cores only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/
# (taken with the kernels as they are in this tree; set an entry to None when its kernel changes)
NCU_TRAFFIC = {
    ("single_step_bf16", "attention_ws_kernel"): 652.2e6 + 83.9e6,
    ("single_step_bf16", "gather_rows_kernel"): 206.1e6 + 153.6e6,
    ("cached_step_bf16", "gather_rows_kernel"): 231.8e6 + 180.0e6,
}
FALLBACK = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return dict(FALLBACK), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                mhz.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = sorted(mhz)[len(mhz) // 2:] if mhz else []
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


# --------------------------------------------------------------------------------------------------
# device workload

class DeviceStep:
    """All buffers of one step resident on the device, plus the calls of the hot path."""

    def __init__(self, ctx, w, seed, device):
        self.ctx, self.w, self.device = ctx, w, device
        g = torch.Generator(device=device)
        g.manual_seed(1000 * w.seed + seed)
        dt = w.torch_dtype
        H, d, R, Lp = w.H, w.d, w.window_rows, w.B + w.window_rows
        rnd = lambda *s: (torch.randn(*s, generator=g, device=device, dtype=torch.float32) * w.sigma).to(dt)
        self.Q, self.K, self.V = rnd(H, R, d), rnd(H, Lp, d), rnd(H, Lp, d)
        self.O = torch.zeros(H, R, d, dtype=dt, device=device)
        self.lse = torch.empty(H, R, dtype=torch.float32, device=device)
        # indicator inputs: every chunk changes by 30 % > eps, so the rule itself recomputes all chunks
        n_el = w.n_c * w.hidden
        self.prev = rnd(w.W * n_el)
        sign = (torch.randint(0, 2, (w.W * n_el,), generator=g, device=device).float() * 2 - 1)
        self.cur = (self.prev.float() * (1 + 0.3 * sign)).to(dt)
        del sign
        self.chunk_off = np.arange(w.W + 1, dtype=np.int64) * n_el
        self.chunk_step = torch.full((w.W,), 5, dtype=torch.int32, device=device)
        self.acc = torch.zeros(w.W, dtype=torch.float32, device=device)
        self.l1rel = torch.empty(w.W, dtype=torch.float32, device=device)
        self.recompute = torch.empty(w.W, dtype=torch.uint8, device=device)
        self.active_ids = torch.empty(w.W, dtype=torch.int32, device=device)
        self.n_active = torch.empty(1, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.q_off, self.vis, self.seg_log, self.seg_phys = wl.prefix_layout(w)
        # compression event: candidates = the first L_k rows of the K/V store, observation queries = the
        # last L_q_obs rows of the last window chunk
        self.L_k = min(w.L_k, Lp)
        self.K_cand, self.V_cand = self.K[:, :self.L_k], self.V[:, :self.L_k]
        self.Q_obs = self.Q[:, R - w.L_q_obs:]
        self.n_keep = min(w.B if w.B > 0 else self.L_k, self.L_k)
        self.score = torch.empty(H, self.L_k, dtype=torch.float32, device=device)
        self.kept_idx = torch.empty(H, self.n_keep, dtype=torch.int32, device=device)
        self.n_kept = torch.empty(1, dtype=torch.int32, device=device)
        self.K_dst = torch.empty(H, self.n_keep, d, dtype=dt, device=device)
        self.V_dst = torch.empty(H, self.n_keep, d, dtype=dt, device=device)
        self.launches_per_step = 2 + 1 + 3 + 2  # decide, attention, score (2 passes, finalize), select, gather

    def bind_inputs(self, t):
        """Point the step at another set of input tensors (same shapes): Q, K, V, cur, prev."""
        self.Q, self.K, self.V, self.cur, self.prev = t["Q"], t["K"], t["V"], t["cur"], t["prev"]
        self.K_cand, self.V_cand = self.K[:, :self.L_k], self.V[:, :self.L_k]
        self.Q_obs = self.Q[:, self.Q.shape[1] - self.w.L_q_obs:]

    def decide(self):
        self.ctx.chunk_decide(self.cur, self.prev, self.chunk_off, self.chunk_step, self.w.warmup_m, self.w.eps,
                              self.acc, l1rel=self.l1rel, recompute=self.recompute, active_ids=self.active_ids,
                              n_active=self.n_active, status=self.status)

    def attention(self):
        self.ctx.chunk_attention(self.Q, self.K, self.V, self.q_off, self.vis, self.seg_log, self.seg_phys,
                                 self.active_ids, self.n_active, self.O, lse=self.lse, status=self.status)

    def score_(self):
        self.ctx.kv_score(self.Q_obs, self.K_cand, lambda_=self.w.lam, pool_k=self.w.pool_k, score=self.score,
                          status=self.status)

    def select_compact(self):
        self.ctx.kv_select_compact(self.score, self.n_keep, self.K_cand, self.V_cand, self.K_dst, self.V_dst,
                                   kept_idx=self.kept_idx, n_kept=self.n_kept, status=self.status)

    STAGES = ("decide", "attention", "score", "select_compact")

    def run(self, events=None):
        for i, fn in enumerate((self.decide, self.attention, self.score_, self.select_compact)):
            if events is not None:
                events[i][0].record()
            fn()
            if events is not None:
                events[i][1].record()


def time_frame_score(step, iters=20):
    """fc_kv_score with one latent frame of observation queries (30 x 52 tokens) instead of 50 tokens: the score
    stage as a dense contraction.  Separate from the timed step; returns (ms per call, L_q)."""
    L_q = min(1560, step.w.n_c)
    R = step.Q.shape[1]
    Q_frame = step.Q[:, R - L_q:]
    score = torch.empty_like(step.score)
    for _ in range(3):
        step.ctx.kv_score(Q_frame, step.K_cand, lambda_=step.w.lam, pool_k=step.w.pool_k, score=score, status=step.status)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(iters):
        step.ctx.kv_score(Q_frame, step.K_cand, lambda_=step.w.lam, pool_k=step.w.pool_k, score=score, status=step.status)
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / iters, L_q


def attention_flops(w, active):
    return w.attention_flops(active)


def run_sweep(step, thresholds, n_steps, peak_tflops):
    """The denoising sweep: per threshold, `n_steps` consecutive steps whose per-chunk change indicator shrinks
    from step to step (u * kappa_s, u ~ U(0,1), kappa_s geometric from 1 to 0.02), so the share of recomputed
    chunks falls from all of them to a few.  Each step runs decide -> attention with the active list staying on
    the device; per step the realised active fraction, the stage times and the attention roofline fraction."""
    w, dev = step.w, step.device
    n_el = w.n_c * w.hidden
    g = torch.Generator(device=dev)
    g.manual_seed(4242)
    sign = (torch.randint(0, 2, (w.W, n_el), generator=g, device=dev, dtype=torch.int8) * 2 - 1)
    prev = step.prev.view(w.W, n_el)
    out = []
    for eps in thresholds:
        step.acc.zero_()
        rows = []
        for s in range(n_steps):
            kappa = 0.02 ** (s / max(n_steps - 1, 1))
            r = torch.rand(w.W, 1, generator=g, device=dev) * kappa
            step.cur.view(w.W, n_el).copy_((prev.float() * (1 + r * sign)).to(prev.dtype))
            step.chunk_step.fill_(s)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            ev[0].record()
            step.ctx.chunk_decide(step.cur, step.prev, step.chunk_off, step.chunk_step, 1, eps, step.acc,
                                  l1rel=step.l1rel, recompute=step.recompute, active_ids=step.active_ids,
                                  n_active=step.n_active, status=step.status)
            ev[1].record()
            step.attention()
            ev[2].record()
            torch.cuda.synchronize()
            n_act = int(step.n_active.item())
            active = step.active_ids[:n_act].cpu().tolist()
            att_ms = ev[1].elapsed_time(ev[2])
            tf = attention_flops(w, active) / (att_ms * 1e-3) / 1e12 if n_act else 0.0
            rows.append({"step": s, "active_fraction": n_act / w.W, "decide_ms": ev[0].elapsed_time(ev[1]),
                         "attention_ms": att_ms, "attention_tflops": tf, "frac": tf / peak_tflops})
        out.append({"eps": eps, "steps": rows})
    del sign
    return out


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a few per-rank timings over all ranks (the slowest rank sets the job's time).
    `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(world, flops_per_rank_step, ms_per_step):
    """Whole-job TFLOP/s of `world` replicas that each do `flops_per_rank_step` per step (weak scaling)."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def time_device(step, steps, warmup, barrier):
    for _ in range(warmup):
        step.run()
    torch.cuda.synchronize()
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in DeviceStep.STAGES]
          for _ in range(steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t0.record()
    for k in range(steps):
        step.run(ev[k])
    t1.record()
    torch.cuda.synchronize()
    barrier()
    total_ms = t0.elapsed_time(t1)
    stage_ms = {name: statistics.mean(ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(steps))
                for i, name in enumerate(DeviceStep.STAGES)}
    return total_ms, stage_ms


def time_e2e(step, steps, warmup, barrier):
    """Same step, but its inputs start in pinned host memory and its results end there.

    Three streams: host-to-device copies of step k+1 run while step k computes (two sets of device input
    buffers), and the results of step k go back while step k+1's inputs are still arriving; the compute of step
    k+1 waits for the read-back of step k, because the output buffers are single.  Every step's copies, both ways,
    are inside the timed region."""
    names = ("Q", "K", "V", "cur", "prev")
    host = {n: getattr(step, n).cpu().pin_memory() for n in names}
    out_host = {"O": torch.empty_like(step.O, device="cpu").pin_memory(),
                "recompute": torch.empty_like(step.recompute, device="cpu").pin_memory(),
                "kept_idx": torch.empty_like(step.kept_idx, device="cpu").pin_memory()}
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())
    sets = [{n: getattr(step, n) for n in names}, {n: torch.empty_like(getattr(step, n)) for n in names}]
    compute = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]     # inputs of a step have landed in set k % 2
    ev_free = [torch.cuda.Event() for _ in range(2)]   # the step that read set k % 2 has finished
    ev_done, ev_out = torch.cuda.Event(), torch.cuda.Event()
    state = {"k": 0}
    for e in ev_free:
        e.record(compute)
    ev_out.record(s_out)

    def one():
        k = state["k"]
        state["k"] = k + 1
        cur = sets[k % 2]
        s_in.wait_event(ev_free[k % 2])
        with torch.cuda.stream(s_in):
            for n in names:
                cur[n].copy_(host[n], non_blocking=True)
            ev_in[k % 2].record(s_in)
        compute.wait_event(ev_in[k % 2])
        compute.wait_event(ev_out)  # the previous step's results have left the output buffers
        step.bind_inputs(cur)
        step.run()
        ev_free[k % 2].record(compute)
        ev_done.record(compute)
        s_out.wait_event(ev_done)
        with torch.cuda.stream(s_out):
            for n, t in out_host.items():
                t.copy_(getattr(step, n), non_blocking=True)
            ev_out.record(s_out)

    for _ in range(max(2, warmup // 2)):
        one()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t0.record(compute)
    for _ in range(steps):
        one()
    compute.wait_event(ev_out)  # the last read-back is inside the timed region
    t1.record(compute)
    torch.cuda.synchronize()
    barrier()
    step.bind_inputs(sets[0])
    return t0.elapsed_time(t1), h2d, d2h


# --------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)

def oracle_sample(w, seed, n_rows):
    """Time the oracle's attention on `n_rows` sampled query rows (all heads) of the workload.
    Returns (seconds, flops evaluated, cores used, description)."""
    import oracle
    Q, K, V = wl.qkv(w, seed)
    q_off, vis, slo, spo = wl.prefix_layout(w)
    rows = wl.sample_rows(w, n_rows, seed)
    if len(rows) > n_rows:
        rows = rows[np.unique(np.linspace(0, len(rows) - 1, n_rows).astype(int))]
    Qb, Kb, Vb = wl.bits(Q), wl.bits(K), wl.bits(V)
    cores = oracle.hardware_threads()
    t = time.perf_counter()
    oracle.chunk_attention(Qb, Kb, Vb, q_off, vis, slo, spo, list(range(w.W)), sample_rows=rows)
    dt = time.perf_counter() - t
    flops = sum(4.0 * w.d * w.H * (w.B + (int(r) // w.n_c + 1) * w.n_c) for r in rows)
    return dt, flops, cores, f"attention oracle on {len(rows)} sampled query rows x {w.H} heads of {w.name}"


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    times, flops = [], 0.0
    n_rows = 48
    for k in range(args.warmup + args.steps):
        dt, fl, cores, desc = oracle_sample(w, k, n_rows)
        if k >= args.warmup:
            times.append(dt)
            flops = fl
    ms = 1e3 * statistics.mean(times)
    value = flops / (ms * 1e-3) / 1e12
    line = {"impl": "reference", "metric": "chunk_attn_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample": desc},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="single_step_bf16", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="fc", choices=["fc", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="also run the 30-step denoising sweep at thresholds 0.05 / 0.1 / 0.2 and add it to the line")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "fc" else args.warmup
    w = wl.CONFIGS[args.config]

    if args.impl == "reference":
        run_reference(args, w)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    import paper_2602_10825_b200 as fc
    from paper_2602_10825_b200 import build as fc_build
    if rank == 0:
        fc_build.build()
    barrier()
    ctx = fc.Context(local_rank)
    step = DeviceStep(ctx, w, seed=rank, device=device)

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, stage_ms = time_device(step, args.steps, args.warmup, barrier)
    clocks = sampler.stop()
    status = int(step.status.item())
    n_active = int(step.n_active.item())
    active = step.active_ids[:n_active].cpu().tolist()
    flops = attention_flops(w, active)

    e2e = None
    if not args.no_e2e:
        e2e_steps = max(2, min(args.steps // 4, 40))
        e2e_ms, h2d, d2h = time_e2e(step, e2e_steps, args.warmup, barrier)
    total_ms, e2e_step_ms = max_over_ranks([total_ms, e2e_ms / e2e_steps if not args.no_e2e else 0.0], dist, device)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        ms_per_step = total_ms / args.steps
        value = job_throughput(world, flops, ms_per_step)
        attn_tflops = flops / (stage_ms["attention"] * 1e-3) / 1e12
        compact_bytes = 4 * step.n_keep * w.d * 2 * w.H
        compact_gbs = compact_bytes / (stage_ms["select_compact"] * 1e-3) / 1e9
        score_gbs = step.L_k * w.d * 2 * w.H / (stage_ms["score"] * 1e-3) / 1e9
        decide_gbs = 2 * step.cur.numel() * 2 / (stage_ms["decide"] * 1e-3) / 1e9
        line = {
            "metric": "chunk_attn_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "H": w.H, "d": w.d, "chunks": w.W, "tokens_per_chunk": w.n_c,
                       "clean_budget": w.B, "active_chunks": active, "candidates": step.L_k, "kept": step.n_keep,
                       "l2": "inputs larger than L2 (K+V %d MB, indicator pair %d MB; L2 126 MB)" % (
                           2 * step.K.numel() * 2 // 2**20, 2 * step.cur.numel() * 2 // 2**20),
                       "parallelism": "replicas" if world > 1 else "single"},
            "stages_ms": stage_ms,
            "roofline": {"bound": "tensor", "achieved": attn_tflops, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": attn_tflops / peaks["bf16_tflops"],
                         "traffic": NCU_TRAFFIC.get((w.name, "attention_ws_kernel")), "kernel": "attention_ws_kernel",
                         "peak_kind": peak_kind + " burst", "frac_of_nominal": attn_tflops / NOMINAL["bf16_tflops"],
                         "frac_of_sustained": attn_tflops / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])},
            "roofline_compact": {"bound": "hbm", "achieved": compact_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": compact_gbs / peaks["hbm_gbs"],
                                 "traffic": NCU_TRAFFIC.get((w.name, "gather_rows_kernel")),
                                 "kernel": "select + gather_rows_kernel (whole fc_kv_select_compact call)",
                                 "peak_kind": peak_kind, "frac_of_nominal": compact_gbs / NOMINAL["hbm_gbs"]},
            "roofline_score": {"bound": "hbm", "achieved": score_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": score_gbs / peaks["hbm_gbs"], "traffic": None,
                               "kernel": "score_tc_kernel passes 1 and 2 + score_finalize_kernel (whole fc_kv_score call); "
                                         "algorithmic bytes = the candidate keys once", "peak_kind": peak_kind},
            "roofline_decide": {"bound": "hbm", "achieved": decide_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": decide_gbs / peaks["hbm_gbs"], "traffic": None,
                                "kernel": "decide_partial_kernel + decide_finalize_kernel (whole fc_chunk_decide call)",
                                "peak_kind": peak_kind},
            "clocks": clocks, "device_status": status,
            "gpu_launches": step.launches_per_step * args.steps,
        }
        if not args.no_e2e:
            line["e2e"] = {"value": job_throughput(world, flops, e2e_step_ms), "unit": "TFLOP/s",
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_step_ms,
                           "overlap": "copies of step k+1 run under the compute of step k (three streams)"}
        if w.dtype == "bf16" and world == 1:
            fr_ms, fr_lq = time_frame_score(step)
            fr_flops = 2 * 2.0 * fr_lq * step.L_k * w.d * w.H  # the logits twice: log-sum-exp pass and mass pass
            fr_tflops = fr_flops / (fr_ms * 1e-3) / 1e12
            line["roofline_score_frame"] = {
                "bound": "tensor", "achieved": fr_tflops, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": fr_tflops / peaks["bf16_tflops"], "traffic": None, "ms": fr_ms, "L_q": fr_lq,
                "kernel": "score_mass_kernel x2 (row statistics, masses) + CUDA-core key statistics and "
                          "finalize (whole fc_kv_score call, outside the timed step); algorithmic FLOPs = "
                          "2 passes x 2 L_q L_k d H", "peak_kind": peak_kind + " burst"}
        if args.sweep:
            line["sweep"] = run_sweep(step, (0.05, 0.1, 0.2), 30, peaks["bf16_tflops"])
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            dt, fl, cores, desc = oracle_sample(w, 0, 1536)
            line["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                                    "sample": desc + f" ({dt:.1f} s)"}
        print(json.dumps(line))
    barrier()
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
