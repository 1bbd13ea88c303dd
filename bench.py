#!/usr/bin/env python
"""Benchmark of the FlowCache hot path on B200: one "step" = decide -> chunk-causal attention ->
score -> top-B select -> gather-compact over one batch of synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the attention work (algorithmic FLOPs of the active
chunks' visible prefixes) divided by the time of the WHOLE step, inputs resident in HBM; `e2e`
is the same with host buffers and the host<->device copies inside the timed region; `roofline`
describes the dominant kernel (attention, tensor-bound) and `roofline_compact` the whole
select + gather call under a real top-B selection (HBM-bound); `cpu_baseline` is the CPU oracle's
attention timed on a sample of query rows bounded by seconds, `cpu_baseline_compress` the oracle's
score + select + compact of the same compression event timed in full.
The default workload is the largest configuration (sweep_bf16: 16 chunks of 6240 tokens all active over a
37440-token clean region, compression 43680 -> 37440).
With --impl reference the oracle itself is the timed program (host cores only).
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
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
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")
CSRC = os.path.join(ROOT, "paper_2602_10825_b200", "csrc")


def ncu_traffic(kernel, workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` on `workload`, from the tracked table
    of ncu captures under profiles/.  A row counts only while the kernel's source file still has the hash the
    capture was taken with; otherwise (or with no row) the answer is None."""
    try:
        rows = [ln.split() for ln in open(TRAFFIC_TABLE) if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None
    for r in rows:
        if len(r) >= 6 and r[0] == kernel and r[1] == workload:
            try:
                digest = hashlib.sha256(open(os.path.join(CSRC, r[2]), "rb").read()).hexdigest()[:16]
            except OSError:
                return None
            return float(r[4]) + float(r[5]) if digest == r[3] else None
    return None


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

    def __init__(self, ctx, w, seed, device, attention_only=False):
        self.ctx, self.w, self.device = ctx, w, device
        g = torch.Generator(device=device)
        g.manual_seed(1000 * w.seed + seed)
        dt = w.torch_dtype
        H, d, R, Lp = w.H, w.d, w.window_rows, w.B + w.window_rows
        rnd = lambda *s: (torch.randn(*s, generator=g, device=device, dtype=torch.float32) * w.sigma).to(dt)
        self.Q, self.K, self.V = rnd(H, R, d), rnd(H, Lp, d), rnd(H, Lp, d)
        self.O = torch.zeros(H, R, d, dtype=dt, device=device)
        self.lse = torch.empty(H, R, dtype=torch.float32, device=device)
        self.active_ids = torch.empty(w.W, dtype=torch.int32, device=device)
        self.n_active = torch.empty(1, dtype=torch.int32, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.q_off, self.vis, self.seg_log, self.seg_phys = wl.prefix_layout(w)
        if attention_only:
            return
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
    the device, then one compression event (score -> select -> compact); per step the realised active fraction,
    the stage times, the attention rate against the sustained matmul rate and the compaction rate."""
    w, dev = step.w, step.device
    n_el = w.n_c * w.hidden
    g = torch.Generator(device=dev)
    g.manual_seed(4242)
    sign = (torch.randint(0, 2, (w.W, n_el), generator=g, device=dev, dtype=torch.int8) * 2 - 1)
    prev = step.prev.view(w.W, n_el)
    hbm = measured_peaks()[0]["hbm_gbs"]
    compact_bytes = 4 * step.n_keep * w.d * step.K.element_size() * w.H
    out = []
    for eps in thresholds:
        step.acc.zero_()
        rows = []
        for s in range(n_steps):
            kappa = 0.02 ** (s / max(n_steps - 1, 1))
            r = torch.rand(w.W, 1, generator=g, device=dev) * kappa
            step.cur.view(w.W, n_el).copy_((prev.float() * (1 + r * sign)).to(prev.dtype))
            step.chunk_step.fill_(s)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            ev[0].record()
            step.ctx.chunk_decide(step.cur, step.prev, step.chunk_off, step.chunk_step, 1, eps, step.acc,
                                  l1rel=step.l1rel, recompute=step.recompute, active_ids=step.active_ids,
                                  n_active=step.n_active, status=step.status)
            ev[1].record()
            step.attention()
            ev[2].record()
            step.score_()
            ev[3].record()
            step.select_compact()
            ev[4].record()
            torch.cuda.synchronize()
            n_act = int(step.n_active.item())
            active = step.active_ids[:n_act].cpu().tolist()
            att_ms, sc_ms = ev[1].elapsed_time(ev[2]), ev[3].elapsed_time(ev[4])
            tf = attention_flops(w, active) / (att_ms * 1e-3) / 1e12 if n_act else 0.0
            gbs = compact_bytes / (sc_ms * 1e-3) / 1e9
            rows.append({"step": s, "active_fraction": n_act / w.W, "decide_ms": ev[0].elapsed_time(ev[1]),
                         "attention_ms": att_ms, "attention_tflops": tf, "frac": tf / peak_tflops,
                         "score_ms": ev[2].elapsed_time(ev[3]), "select_compact_ms": sc_ms, "compact_gbs": gbs,
                         "compact_frac": gbs / hbm})
        out.append({"eps": eps, "steps": rows})
    del sign
    return out


def run_streaming(ctx, device, n_chunks, steps_per_chunk=None):
    """The streaming configuration as a sequence: chunks generated one after another (keys drifting as an AR(1)
    process), each denoised for S steps of attention over [history | itself] with the importance of the history
    accumulated over those steps, then scored, selected and compacted back to the budget (identity while the
    history still fits).  Returns per-chunk stage times and the means over the chunks that really compressed."""
    w = wl.CONFIGS["streaming_bf16"]
    H, d, n_c, B = w.H, w.d, w.n_c, w.B
    S = steps_per_chunk or w.n_steps
    g = torch.Generator(device=device)
    g.manual_seed(1000 * w.seed + 77)
    rnd = lambda *s: torch.randn(*s, generator=g, device=device, dtype=torch.float32)
    stores = [[torch.zeros(H, B + n_c, d, dtype=torch.bfloat16, device=device) for _ in range(2)] for _ in range(2)]
    state = rnd(H, n_c, d)
    O = torch.zeros(H, n_c, d, dtype=torch.bfloat16, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    one = torch.ones(1, dtype=torch.int32, device=device)
    zero_id = torch.zeros(1, dtype=torch.int32, device=device)
    q_off = np.array([0, n_c], np.int32)
    L_hist, cur, per_chunk = 0, 0, []
    rho = 0.98
    for c in range(n_chunks):
        K, V = stores[cur]
        K[:, L_hist:L_hist + n_c] = (state * w.sigma).to(torch.bfloat16)
        V[:, L_hist:L_hist + n_c] = (rnd(H, n_c, d) * w.sigma).to(torch.bfloat16)
        state = rho * state + (1 - rho * rho) ** 0.5 * rnd(H, n_c, d)
        L_all = L_hist + n_c
        vis, slo, spo = np.array([L_all], np.int32), np.array([0, L_all], np.int32), np.array([0], np.int32)
        Qs = [(rnd(H, n_c, d) * w.sigma).to(torch.bfloat16) for _ in range(S)]
        # the stores are [H, B + n_c, d]: the first L_all rows of every head are passed as strided views
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        att_ms = sc_ms = 0.0
        acc_c = torch.zeros(H, L_all, dtype=torch.float32, device=device)
        score_c = torch.empty(H, L_all, dtype=torch.float32, device=device)
        for s_ in range(S):
            ev[0].record()
            ctx.chunk_attention(Qs[s_], K, V, q_off, vis, slo, spo, zero_id, one, O, status=status)
            ev[1].record()
            ctx.kv_score(Qs[s_][:, n_c - w.L_q_obs:], K[:, :L_all], lambda_=w.lam, pool_k=w.pool_k, imp_accum=acc_c,
                         accum_phase=2 if s_ == S - 1 else 1, n_steps=S, score=score_c, status=status)
            ev[2].record()
            torch.cuda.synchronize()
            att_ms += ev[0].elapsed_time(ev[1])
            sc_ms += ev[1].elapsed_time(ev[2])
        K2, V2 = stores[cur ^ 1]
        n_keep = min(B, L_all)
        ev[2].record()
        ctx.kv_select_compact(score_c, B, K[:, :L_all], V[:, :L_all], K2[:, :n_keep], V2[:, :n_keep], status=status)
        ev[3].record()
        torch.cuda.synchronize()
        per_chunk.append({"chunk": c, "candidates": L_all, "kept": n_keep, "attention_ms": att_ms, "score_ms": sc_ms,
                          "select_compact_ms": ev[2].elapsed_time(ev[3]),
                          "attention_tflops": S * 4.0 * d * H * n_c * L_all / (att_ms * 1e-3) / 1e12,
                          "compact_gbs": 4 * n_keep * d * 2 * H / (ev[2].elapsed_time(ev[3]) * 1e-3) / 1e9})
        L_hist, cur = n_keep, cur ^ 1
    real = [r for r in per_chunk if r["candidates"] > B]
    mean = lambda k: statistics.mean(r[k] for r in real) if real else None
    return {"workload": w.name, "chunks": n_chunks, "steps_per_chunk": S, "compressions": len(real),
            "mean_over_compressing_chunks": {k: mean(k) for k in ("attention_ms", "score_ms", "select_compact_ms",
                                                                  "attention_tflops", "compact_gbs")},
            "device_status": int(status.item()), "per_chunk": per_chunk}


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
    per_stage = {name: [ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(steps)]
                 for i, name in enumerate(DeviceStep.STAGES)}
    stage_ms = {name: statistics.mean(v) for name, v in per_stage.items()}
    stage_ms["median"] = {name: statistics.median(v) for name, v in per_stage.items()}
    stage_ms["best"] = {name: min(v) for name, v in per_stage.items()}
    return total_ms, stage_ms


def time_e2e(step, steps, warmup, barrier):
    """Same step, but its inputs start in pinned host memory and its results end there.

    Three streams and two sets of device buffers for inputs AND outputs: the host-to-device copies of step k+1 and
    the read-back of step k - 1 both run while step k computes.  Every step's copies, both ways, are inside the timed
    region (the last read-back is waited for before the closing event)."""
    names = ("Q", "K", "V", "cur", "prev")
    out_names = ("O", "recompute", "kept_idx")
    host = {n: getattr(step, n).cpu().pin_memory() for n in names}
    out_host = {n: torch.empty_like(getattr(step, n), device="cpu").pin_memory() for n in out_names}
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in out_host.values())
    sets = [{n: getattr(step, n) for n in names}, {n: torch.empty_like(getattr(step, n)) for n in names}]
    outs = [{n: getattr(step, n) for n in out_names}, {n: torch.empty_like(getattr(step, n)) for n in out_names}]
    compute = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]     # inputs of a step have landed in set k % 2
    ev_free = [torch.cuda.Event() for _ in range(2)]   # the step that read set k % 2 has finished
    ev_done = [torch.cuda.Event() for _ in range(2)]   # the step that wrote output set k % 2 has finished
    ev_out = [torch.cuda.Event() for _ in range(2)]    # output set k % 2 has been read back
    state = {"k": 0}
    for e in ev_free:
        e.record(compute)
    for e in ev_out:
        e.record(s_out)

    def one():
        k = state["k"]
        state["k"] = k + 1
        cur, out = sets[k % 2], outs[k % 2]
        s_in.wait_event(ev_free[k % 2])
        with torch.cuda.stream(s_in):
            for n in names:
                cur[n].copy_(host[n], non_blocking=True)
            ev_in[k % 2].record(s_in)
        compute.wait_event(ev_in[k % 2])
        compute.wait_event(ev_out[k % 2])  # the results of step k - 2 have left this output set
        step.bind_inputs(cur)
        for n in out_names:
            setattr(step, n, out[n])
        step.run()
        ev_free[k % 2].record(compute)
        ev_done[k % 2].record(compute)
        s_out.wait_event(ev_done[k % 2])
        with torch.cuda.stream(s_out):
            for n in out_names:
                out_host[n].copy_(out[n], non_blocking=True)
            ev_out[k % 2].record(s_out)

    for _ in range(max(2, warmup // 2)):
        one()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t0.record(compute)
    for _ in range(steps):
        one()
    for e in ev_out:
        compute.wait_event(e)  # the last read-backs are inside the timed region
    t1.record(compute)
    torch.cuda.synchronize()
    barrier()
    step.bind_inputs(sets[0])
    for n in out_names:
        setattr(step, n, outs[0][n])
    return t0.elapsed_time(t1), h2d, d2h


# --------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline legs and --impl reference)

class OracleAttention:
    """The oracle's chunk-causal attention on sampled query rows of the workload (all chunks active, all heads,
    the full visible prefix of each row).  Inputs are drawn once; every call takes its own sample of rows."""

    def __init__(self, w):
        import oracle
        oracle.build()
        self.oracle, self.w = oracle, w
        Q, K, V = wl.qkv(w)
        self.Q, self.K, self.V = wl.bits(Q), wl.bits(K), wl.bits(V)
        self.q_off, self.vis, self.slo, self.spo = wl.prefix_layout(w)
        self.cores = oracle.hardware_threads()

    def run(self, n_rows, seed):
        """Returns (seconds, algorithmic FLOPs of the rows evaluated, rows)."""
        w = self.w
        # distinct rows drawn uniformly over the window: the sample's size is exact
        pool = torch.randperm(w.window_rows, generator=torch.Generator().manual_seed(1000 * w.seed + seed))[:n_rows]
        rows = np.sort(pool.numpy().astype(np.int32))
        t = time.perf_counter()
        self.oracle.chunk_attention(self.Q, self.K, self.V, self.q_off, self.vis, self.slo, self.spo,
                                    list(range(w.W)), sample_rows=rows)
        dt = time.perf_counter() - t
        flops = sum(4.0 * w.d * w.H * (w.B + (int(r) // w.n_c + 1) * w.n_c) for r in rows)
        return dt, flops, len(rows)

    def rows_for(self, seconds, probe_rows=4):
        """How many rows the oracle evaluates in about `seconds` on this machine (from a small probe)."""
        dt, _, n = self.run(probe_rows, 12345)
        return max(probe_rows, min(8192, int(n * seconds / max(dt, 1e-3))))


def oracle_compress(w):
    """The oracle's compression event of the workload, in full: score (Eqs. 9-12), top-B, compaction.
    Returns (seconds score, seconds select+compact, bytes kept and moved, cores)."""
    import oracle
    oracle.build()
    Q_obs, K, V = wl.candidates(w)
    Qb, Kb, Vb = wl.bits(Q_obs), wl.bits(K), wl.bits(V)
    t0 = time.perf_counter()
    sc = oracle.kv_score(Qb, Kb, lambda_=w.lam, pool_k=w.pool_k)
    t1 = time.perf_counter()
    oracle.kv_select_compact(sc["score"], w.B if w.B > 0 else w.L_k, Kb, Vb)
    t2 = time.perf_counter()
    n_keep = min(w.B if w.B > 0 else w.L_k, w.L_k)
    return t1 - t0, t2 - t1, 4 * n_keep * w.d * 2 * w.H, oracle.hardware_threads()


def config_dict(w, world):
    """The `config` object of the JSON line; both arms print the same one."""
    Lp = w.B + w.window_rows
    L_k = min(w.L_k, Lp)
    n_keep = min(w.B if w.B > 0 else L_k, L_k)
    kv_mb = 2 * w.H * Lp * w.d * 2 // 2**20
    ind_mb = 2 * w.W * w.n_c * w.hidden * 2 // 2**20
    return {"workload": w.name, "H": w.H, "d": w.d, "chunks": w.W, "tokens_per_chunk": w.n_c, "clean_budget": w.B,
            "active_chunks": list(range(w.W)), "candidates": L_k, "kept": n_keep,
            "selection": "identity (budget = cache length)" if n_keep == L_k else "top-B radix select",
            "l2": "inputs larger than L2 (K+V %d MB, indicator pair %d MB; L2 126 MB)" % (kv_mb, ind_mb),
            "parallelism": "replicas" if world > 1 else "single"}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    oa = OracleAttention(w)
    n_rows = oa.rows_for(0.5)  # a step of about half a second, so that --steps K --warmup W ends within minutes
    times, flops = [], 0.0
    for k in range(args.warmup + args.steps):
        dt, fl, n = oa.run(n_rows, k)
        if k >= args.warmup:
            times.append(dt)
            flops = fl
    ms = 1e3 * statistics.mean(times)
    value = flops / (ms * 1e-3) / 1e12
    desc = f"attention oracle on {n_rows} sampled query rows x {w.H} heads of {w.name} per step"
    line = {"impl": "reference", "metric": "chunk_attn_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, world),
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oa.cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# measurements outside the timed step

def time_calls(fn, iters=20, warm=3):
    """Mean CUDA-event time in ms of `fn()` over `iters` calls after `warm` untimed ones."""
    for _ in range(warm):
        fn()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(iters):
        fn()
    t1.record()
    torch.cuda.synchronize()
    return t0.elapsed_time(t1) / iters


def time_cache_apply(step, iters=10):
    """fc_chunk_cache_apply over the step's indicator-sized tensors with every other chunk served from the cache.
    Returns (ms per call, bytes moved per call)."""
    w = step.w
    y = torch.empty_like(step.cur)
    cache = torch.zeros_like(step.cur)
    flags = torch.tensor([c % 2 for c in range(w.W)], dtype=torch.uint8, device=step.device)
    ms = time_calls(lambda: step.ctx.chunk_cache_apply(step.cur, y, cache, step.chunk_off, flags), iters)
    return ms, 3 * step.cur.numel() * step.cur.element_size()


def time_token_map_attention(step, iters=5):
    """fc_chunk_attention of all chunks with the K/V store read through a per-head token map (tile::gather4 loads)
    instead of the segment table: the clean region is a sorted random subset of the candidate rows, as a top-B
    selection leaves it, the window follows.  Returns ms per call."""
    w, dev = step.w, step.device
    g = torch.Generator(device=dev)
    g.manual_seed(99)
    n_clean = step.n_keep if w.B > 0 else 0
    parts = []
    if n_clean:
        pick = torch.rand(w.H, step.L_k, generator=g, device=dev).argsort(dim=1)[:, :n_clean].sort(dim=1).values
        parts.append(pick.to(torch.int32))
    parts.append((w.B + torch.arange(w.window_rows, device=dev, dtype=torch.int32)).repeat(w.H, 1))
    tok = torch.cat(parts, dim=1).contiguous()
    act = torch.arange(w.W, dtype=torch.int32, device=dev)
    n_act = torch.full((1,), w.W, dtype=torch.int32, device=dev)
    fn = lambda: step.ctx.chunk_attention(step.Q, step.K, step.V, step.q_off, step.vis, None, None, act, n_act, step.O,
                                          kv_token_index=tok, impl=2, status=step.status)
    return time_calls(fn, iters, 2)


def time_single_step_attention(ctx, device, iters=20, head_dim=128):
    """The attention kernel alone on the single-step configuration (16 heads, 4 x 6240 tokens, no clean region):
    short enough to run at burst clocks.  head_dim = 64: the same hidden width as 32 heads of 64.
    Returns (ms, algorithmic FLOPs)."""
    w = wl.CONFIGS["single_step_bf16"]
    if head_dim != w.d:
        w = dataclasses.replace(w, name=f"{w.name}_d{head_dim}", H=w.H * w.d // head_dim, d=head_dim)
    st = DeviceStep(ctx, w, seed=0, device=device, attention_only=True)
    st.n_active.fill_(w.W)
    st.active_ids.copy_(torch.arange(w.W, dtype=torch.int32, device=device))
    ms = time_calls(st.attention, iters)
    return ms, w.attention_flops(range(w.W))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="sweep_bf16", choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="fc", choices=["fc", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the measurements taken outside the timed step (frame-level score, cache apply, ...)")
    ap.add_argument("--sweep", action="store_true",
                    help="also run the 30-step denoising sweep at thresholds 0.05 / 0.1 / 0.2 and add it to the line")
    ap.add_argument("--streaming", type=int, default=0, metavar="CHUNKS",
                    help="also generate CHUNKS chunks in sequence (importance accumulated over the chunk's steps, "
                         "compression after every chunk) and add the per-chunk stage times to the line")
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
    single = single_d64 = None
    if world == 1 and w.dtype == "bf16" and w.name != "single_step_bf16" and not args.no_extras:
        single = time_single_step_attention(ctx, device)  # before the long loop: at burst clocks, as a kernel timed alone
        single_d64 = time_single_step_attention(ctx, device, head_dim=64)
    step = DeviceStep(ctx, w, seed=rank, device=device)

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, stage_ms = time_device(step, args.steps, args.warmup, barrier)
    clocks = sampler.stop()
    status = int(step.status.item())
    n_active = int(step.n_active.item())
    active = step.active_ids[:n_active].cpu().tolist()
    flops = attention_flops(w, active)

    e2e_ms, e2e_steps, h2d, d2h = 0.0, 1, 0, 0
    if not args.no_e2e:
        # as many steps as the device-timed loop (the first step's input copy and the last read-back are exposed:
        # about 65 + 11 ms on the default workload, amortised over the steps)
        e2e_steps = max(2, min(args.steps, 100))
        e2e_ms, h2d, d2h = time_e2e(step, e2e_steps, args.warmup, barrier)
    total_ms, e2e_step_ms = max_over_ranks([total_ms, e2e_ms / e2e_steps], dist, device)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        ms_per_step = total_ms / args.steps
        value = job_throughput(world, flops, ms_per_step)
        attn_tflops = flops / (stage_ms["attention"] * 1e-3) / 1e12
        es = 2 if w.dtype == "bf16" else 4
        compact_bytes = 4 * step.n_keep * w.d * es * w.H
        compact_gbs = compact_bytes / (stage_ms["select_compact"] * 1e-3) / 1e9
        score_gbs = step.L_k * w.d * es * w.H / (stage_ms["score"] * 1e-3) / 1e9
        decide_gbs = 2 * step.cur.numel() * es / (stage_ms["decide"] * 1e-3) / 1e9
        # a kernel that runs for tens of milliseconds inside a loop of seconds is held by the power cap: its
        # denominator is the sustained matmul rate; a kernel of a few milliseconds is compared with the burst rate
        long_step = stage_ms["attention"] * args.steps > 1000.0
        tensor_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) if long_step else peaks["bf16_tflops"]
        real_selection = step.n_keep < step.L_k
        cfg = config_dict(w, world)
        cfg["active_chunks"] = active
        line = {
            "metric": "chunk_attn_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": cfg,
            "stages_ms": stage_ms,
            "roofline": {"bound": "tensor", "achieved": attn_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                         "frac": attn_tflops / tensor_peak,
                         "traffic": ncu_traffic("attention_ws_kernel", w.name), "kernel": "attention_ws_kernel",
                         "peak_kind": peak_kind + (" sustained (the kernel runs inside a loop of seconds)" if long_step
                                                   else " burst"),
                         "frac_of_burst": attn_tflops / peaks["bf16_tflops"],
                         "frac_of_nominal": attn_tflops / NOMINAL["bf16_tflops"],
                         "frac_of_sustained": attn_tflops / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])},
            "roofline_compact": {"bound": "hbm", "achieved": compact_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": compact_gbs / peaks["hbm_gbs"],
                                 "traffic": ncu_traffic("gather_rows_kernel", w.name),
                                 "kernel": ("select_topb_kernel" if real_selection else "select_identity_kernel")
                                           + " + gather_rows_kernel (whole fc_kv_select_compact call; traffic: the gather)",
                                 "peak_kind": peak_kind, "frac_of_nominal": compact_gbs / NOMINAL["hbm_gbs"]},
            "roofline_score": {"bound": "hbm", "achieved": score_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": score_gbs / peaks["hbm_gbs"], "traffic": ncu_traffic("score_tc_kernel", w.name),
                               "kernel": "score_tc_kernel passes 1 and 2 + score_finalize_kernel (whole fc_kv_score call); "
                                         "algorithmic bytes = the candidate keys once", "peak_kind": peak_kind},
            "roofline_decide": {"bound": "hbm", "achieved": decide_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": decide_gbs / peaks["hbm_gbs"],
                                "traffic": ncu_traffic("decide_partial_kernel", w.name),
                                "kernel": "decide_partial_kernel + decide_finalize_kernel (whole fc_chunk_decide call)",
                                "peak_kind": peak_kind},
            "clocks": clocks, "device_status": status,
            "gpu_launches": step.launches_per_step * args.steps,
        }
        if not args.no_e2e:
            line["e2e"] = {"value": job_throughput(world, flops, e2e_step_ms), "unit": "TFLOP/s",
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_step_ms,
                           "overlap": "the input copies of step k+1 and the read-back of step k-1 run under the compute of step k (three streams, two sets of device buffers)"}
        if w.dtype == "bf16" and world == 1 and not args.no_extras:
            fr_ms, fr_lq = time_frame_score(step)
            fr_flops = 2 * 2.0 * fr_lq * step.L_k * w.d * w.H  # the logits twice: log-sum-exp pass and mass pass
            fr_tflops = fr_flops / (fr_ms * 1e-3) / 1e12
            line["roofline_score_frame"] = {
                "bound": "tensor", "achieved": fr_tflops, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": fr_tflops / peaks["bf16_tflops"], "traffic": None, "ms": fr_ms, "L_q": fr_lq,
                "kernel": "score_mass_kernel x2 (row statistics, masses) + CUDA-core key statistics and "
                          "finalize (whole fc_kv_score call, outside the timed step); algorithmic FLOPs = "
                          "2 passes x 2 L_q L_k d H", "peak_kind": peak_kind + " burst"}
            # the memory-bound calls again, timed back to back outside the step: what the copy rate they are compared
            # with was measured as (a short kernel alone), without the clocks and cache state the 100 ms attention
            # kernel leaves behind inside the step
            for key, fn, nbytes in (("roofline_compact", step.select_compact, compact_bytes),
                                    ("roofline_score", step.score_, step.L_k * w.d * es * w.H),
                                    ("roofline_decide", step.decide, 2 * step.cur.numel() * es)):
                a_ms = time_calls(fn, 20)
                a_gbs = nbytes / (a_ms * 1e-3) / 1e9
                line[key]["alone"] = {"ms": a_ms, "achieved": a_gbs, "frac": a_gbs / peaks["hbm_gbs"],
                                      "frac_of_nominal": a_gbs / NOMINAL["hbm_gbs"],
                                      "how": "the same call, 20 times back to back outside the timed step"}
            ca_ms, ca_bytes = time_cache_apply(step)
            ca_gbs = ca_bytes / (ca_ms * 1e-3) / 1e9
            line["roofline_cache_apply"] = {
                "bound": "hbm", "achieved": ca_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ca_gbs / peaks["hbm_gbs"], "traffic": ncu_traffic("cache_apply_kernel", w.name), "ms": ca_ms,
                "kernel": "cache_apply_kernel (fc_chunk_cache_apply, outside the timed step, every other chunk served "
                          "from the cache); algorithmic bytes = 3 x elements x element size", "peak_kind": peak_kind}
            score2 = torch.empty_like(step.score)
            base_ms = time_calls(lambda: step.ctx.kv_score(step.Q_obs, step.K_cand, lambda_=w.lam, pool_k=w.pool_k,
                                                           score=score2, status=step.status), 5, 2)
            rt_ms = time_calls(lambda: step.ctx.kv_score(step.Q_obs, step.K_cand, lambda_=w.lam, pool_k=w.pool_k,
                                                         score=score2, red_mode=1, status=step.status), 5, 2)
            rt_flops = 2.0 * step.L_k * step.L_k * w.d * w.H
            rt_tf = rt_flops / ((rt_ms - base_ms) * 1e-3) / 1e12
            line["roofline_red_tiled"] = {
                "bound": "tensor", "achieved": rt_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": rt_tf / peaks["bf16_tflops"], "traffic": ncu_traffic("red_tiled_kernel", w.name),
                "ms": rt_ms - base_ms, "call_ms": rt_ms,
                "kernel": "red_tiled_kernel + key_inv_norm_kernel (red_mode = tiled: the cosine-similarity matrix in "
                          "128 x 128 tcgen05 tiles, never stored); time = fc_kv_score in tiled mode minus the same call "
                          "in mean-key mode; FLOPs = 2 L_k^2 d H, the dense work the mean-key identity avoids: "
                          "reported apart, not part of the score stage's figure", "peak_kind": peak_kind + " burst"}
            tm_ms = time_token_map_attention(step)
            tm_tf = w.attention_flops(range(w.W)) / (tm_ms * 1e-3) / 1e12
            line["attention_token_map"] = {
                "bound": "tensor", "achieved": tm_tf, "peak": tensor_peak, "unit": "TFLOP/s", "frac": tm_tf / tensor_peak,
                "ms": tm_ms, "segment_table_ms": stage_ms["attention"],
                "kernel": "attention_ws_kernel<D, gather> (all chunks active, K/V rows fetched by tile::gather4 through a "
                          "per-head token map; outside the timed step)", "peak_kind": peak_kind}
            if single is not None:
                a_ms, a_flops = single
                a_tf = a_flops / (a_ms * 1e-3) / 1e12
                line["attention_single_step_bf16"] = {
                    "bound": "tensor", "achieved": a_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": a_tf / peaks["bf16_tflops"], "ms": a_ms, "traffic": ncu_traffic("attention_ws_kernel", "single_step_bf16"),
                    "kernel": "attention_ws_kernel timed alone (20 launches back to back) on single_step_bf16: "
                              "16 heads, 4 chunks of 6240 tokens, all active, no clean region", "peak_kind": peak_kind + " burst"}
            if single_d64 is not None:
                a_ms, a_flops = single_d64
                a_tf = a_flops / (a_ms * 1e-3) / 1e12
                line["attention_single_step_bf16_d64"] = {
                    "bound": "tensor", "achieved": a_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": a_tf / peaks["bf16_tflops"], "ms": a_ms, "traffic": None,
                    "kernel": "attention_ws_kernel<64> timed alone (20 launches back to back): the single-step shape with "
                              "32 heads of 64 instead of 16 of 128 (half the FLOPs per exponential)",
                    "peak_kind": peak_kind + " burst"}
        if args.sweep:
            line["sweep"] = run_sweep(step, (0.05, 0.1, 0.2), 30, peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
        if args.streaming > 0:
            line["streaming"] = run_streaming(ctx, device, args.streaming)
        if world == 1 and not args.no_cpu_baseline:
            oa = OracleAttention(w)
            n_rows = oa.rows_for(18.0)
            dt, fl, n = oa.run(n_rows, 0)
            line["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oa.cores, "kind": "oracle",
                                    "sample": f"attention oracle on {n} uniformly sampled query rows x {w.H} heads of "
                                              f"{w.name}, full visible prefix each ({dt:.1f} s)"}
            del oa
            t_sc, t_sel, nbytes, cores = oracle_compress(w)
            line["cpu_baseline_compress"] = {
                "value": nbytes / (t_sc + t_sel) / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                "sample": f"oracle score + select + compact of the whole compression event of {w.name} "
                          f"({w.H} heads, {step.L_k} -> {step.n_keep} tokens): score {t_sc:.2f} s, select + compact "
                          f"{t_sel:.2f} s; bytes = K and V rows kept, read and written"}
        print(json.dumps(line))
    barrier()
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
