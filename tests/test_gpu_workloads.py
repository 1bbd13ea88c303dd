"""The streaming and the sweep workloads end to end on the GPU against the CPU oracle, at sizes the oracle
finishes in seconds: same chunk counts, step counts, thresholds and key statistics as the full configurations,
fewer heads and shorter chunks (still several 128-token tiles with ragged tails).

Bars as elsewhere: decisions and kept indices bit-exact (the selection is fed the same fp32 scores on both
sides), compacted rows byte-exact, bf16 attention within max-abs 1e-2 / relative-L2 1e-2, scores within 1e-4
of the row maximum.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2602_10825_b200 as fc
    from paper_2602_10825_b200 import build as fc_build
    fc_build.build()
    c = fc.Context(0)
    yield c
    c.close()


def i32(x):
    return torch.as_tensor(np.asarray(x), dtype=torch.int32).cuda()


def _check_attention(got, want, atol=1e-2, rel=1e-2):
    assert np.abs(got - want).max() <= atol
    assert np.linalg.norm(got - want) <= rel * np.linalg.norm(want)


def test_streaming_generation_with_compression_after_every_chunk(ctx):
    # config 4 in small: chunks generated one after another, each denoised for S steps while attending to
    # [history | itself]; the importance is accumulated over the chunk's steps; after the chunk the history is
    # scored, the top B kept and compacted.  The first chunks fill the budget (identity), the rest compress.
    full = wl.CONFIGS["streaming_bf16"]
    H, d, n_c, B, n_chunks, S = 2, full.d, 328, 900, 7, full.n_steps
    keys = list(wl.ar1_keys(H, n_chunks, n_c, d, seed=full.seed, sigma=full.sigma))
    hist_K = torch.empty((H, 0, d), dtype=torch.bfloat16)
    hist_V = torch.empty((H, 0, d), dtype=torch.bfloat16)
    n_compress = 0
    for c in range(n_chunks):
        K_c = keys[c]
        V_c = wl.normal((H, n_c, d), 7000 + c, full.sigma, torch.bfloat16)
        K_all, V_all = torch.cat([hist_K, K_c], 1).contiguous(), torch.cat([hist_V, V_c], 1).contiguous()
        L_hist, L_all = hist_K.shape[1], hist_K.shape[1] + n_c
        q_off, vis = np.array([0, n_c], np.int32), np.array([L_all], np.int32)
        slo = np.array([0, L_hist, L_all] if L_hist else [0, L_all], np.int32)
        spo = np.array([0, L_hist] if L_hist else [0], np.int32)
        acc_g = torch.zeros((H, L_all), device="cuda")
        acc_o = np.zeros((H, L_all), np.float64)
        Kg, Vg = K_all.cuda(), V_all.cuda()
        for s in range(S):
            Q = wl.normal((H, n_c, d), 8000 + 10 * c + s, full.sigma, torch.bfloat16)
            O = torch.zeros((H, n_c, d), dtype=torch.bfloat16, device="cuda")
            ctx.chunk_attention(Q.cuda(), Kg, Vg, q_off, vis, slo, spo, i32([0]), i32([1]), O)
            rows = wl.sample_rows(wl.Workload("x", "bf16", H=H, d=d, W=1, n_c=n_c, B=0, L_k=0, seed=c), 6, s)
            O_want, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K_all), wl.bits(V_all), q_off, vis, slo, spo, [0],
                                               sample_rows=rows)
            _check_attention(O.double().cpu().numpy()[:, rows], O_want)
            Q_obs = Q[:, n_c - full.L_q_obs:].contiguous()
            phase = 2 if s == S - 1 else 1
            want = oracle.kv_score(wl.bits(Q_obs), wl.bits(K_all), lambda_=full.lam, pool_k=full.pool_k,
                                   imp_accum=acc_o, accum_phase=phase, n_steps=S)
            got = ctx.kv_score(Q_obs.cuda(), Kg, lambda_=full.lam, pool_k=full.pool_k, imp_accum=acc_g,
                               accum_phase=phase, n_steps=S)
        torch.cuda.synchronize()
        score = got["score"].cpu().numpy()
        assert np.abs(score - want["score"]).max() <= 1e-4 * np.abs(want["score"]).max()
        sel = ctx.kv_select_compact(got["score"], B, Kg, Vg)
        want_sel = oracle.kv_select_compact(score, B, wl.bits(K_all), wl.bits(V_all))
        torch.cuda.synchronize()
        assert np.array_equal(sel["kept_idx"].cpu().numpy(), want_sel["kept_idx"])
        assert np.array_equal(wl.bits(sel["K_dst"].cpu()), want_sel["K_dst"])
        assert np.array_equal(wl.bits(sel["V_dst"].cpu()), want_sel["V_dst"])
        if L_all <= B:  # fill phase: nothing is dropped
            assert np.array_equal(want_sel["kept_idx"], np.tile(np.arange(L_all, dtype=np.int32), (H, 1)))
        else:
            n_compress += 1
            assert sel["kept_idx"].shape[1] == B
        hist_K, hist_V = sel["K_dst"].cpu(), sel["V_dst"].cpu()
    assert n_compress >= 4


@pytest.mark.parametrize("eps", [0.05, 0.1, 0.2])
def test_denoising_sweep_decisions_and_attention_of_the_active_chunks(ctx, eps):
    # config 5 in small: 16 chunks, 30 steps, the change indicator shrinking from step to step so that the
    # share of recomputed chunks falls from all of them to a few; decisions bit-exact at every step, attention
    # of exactly the active chunks checked at the first step, in the middle and at the end.
    full = wl.CONFIGS["sweep_bf16"]
    w = wl.Workload("sweep_small", "bf16", H=2, d=full.d, W=full.W, n_c=200, B=456, L_k=656, seed=full.seed,
                    sigma=full.sigma, D=256)
    n_el = w.n_c * w.hidden
    off = np.arange(w.W + 1, dtype=np.int64) * n_el
    targets = wl.sweep_targets(full.n_steps, w.W, full.seed).numpy()
    Q, K, V = wl.qkv(w)
    q_off, vis, slo, spo = wl.prefix_layout(w)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    O0 = wl.normal((w.H, w.window_rows, w.d), 77, 1.0, torch.bfloat16)
    acc_o = np.zeros(w.W, np.float32)
    acc_g = torch.zeros(w.W, device="cuda")
    fractions = []
    min_margin = np.inf
    for s in range(full.n_steps):
        step = np.full(w.W, s, np.int32)
        target = targets[s].copy()
        for _ in range(8):  # guard band: a draw that lands a chunk on the threshold is nudged away from it
            cur, prev = wl.indicator_pair(w.W, n_el, target, 5000 + s)
            want = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), off, step, 1, eps, acc_o)
            margin = np.abs(acc_o + want["l1rel"] - eps)
            if s == 0 or margin.min() > 1e-3 * eps:
                break
            target[margin <= 1e-3 * eps] *= 1.03
        if s >= 1:
            min_margin = min(min_margin, float(margin.min()))
        got = ctx.chunk_decide(cur.cuda(), prev.cuda(), off, i32(step), 1, eps, acc_g)
        torch.cuda.synchronize()
        assert got["recompute"].cpu().numpy().tolist() == want["recompute"].tolist(), f"step {s}"
        assert got["active_ids"].cpu().numpy()[:want["n_active"]].tolist() == want["active_ids"].tolist()
        acc_o = want["acc"]
        active = want["active_ids"].tolist()
        fractions.append(len(active) / w.W)
        if s in (0, full.n_steps // 2, full.n_steps - 1):
            O = O0.cuda().clone()
            ctx.chunk_attention(Qg, Kg, Vg, q_off, vis, slo, spo, got["active_ids"], got["n_active"], O)
            torch.cuda.synchronize()
            rows = wl.sample_rows(w, 16, s)
            rows = rows[np.isin(rows // w.n_c, active)]
            if len(rows):
                O_want, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, active,
                                                   sample_rows=rows)
                _check_attention(O.double().cpu().numpy()[:, rows], O_want)
            for c in range(w.W):  # chunks served from cache keep their outputs bit for bit
                if c not in active:
                    assert torch.equal(O[:, q_off[c]:q_off[c + 1]].cpu(), O0[:, q_off[c]:q_off[c + 1]])
    assert min_margin > 1e-3 * eps, f"a step came within {min_margin} of eps; change the seed"
    assert fractions[0] == 1.0 and fractions[-1] <= 0.5 and min(fractions) < max(fractions)


@pytest.mark.parametrize("eps", [0.1, 0.15])
def test_blocks_at_staggered_noise_levels(ctx, eps):
    # the second model family in small: five blocks in flight, block i two denoising steps behind block i - 1, four
    # warm-up steps per block (so at any step some blocks are forced, some decide by threshold), a clean overlap
    # region in front; decisions bit-exact at every step, attention of the active blocks at three of them
    full = wl.CONFIGS["skyreels_bf16"]
    w = wl.Workload("blocks_small", "bf16", H=2, d=full.d, W=full.W, n_c=344, B=344, L_k=688, seed=full.seed,
                    sigma=full.sigma, D=192, eps=eps, warmup_m=full.warmup_m)
    n_el = w.n_c * w.hidden
    off = np.arange(w.W + 1, dtype=np.int64) * n_el
    Q, K, V = wl.qkv(w)
    q_off, vis, slo, spo = wl.prefix_layout(w)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    O0 = wl.normal((w.H, w.window_rows, w.d), 78, 1.0, torch.bfloat16)
    acc_o = np.zeros(w.W, np.float32)
    acc_g = torch.zeros(w.W, device="cuda")
    n_steps, lag = 14, 2
    n_forced = n_reused = 0
    for s in range(n_steps):
        step = np.maximum(s - lag * np.arange(w.W), 0).astype(np.int32)
        target = wl.uniform((w.W,), 900 + s, 0.0, 0.12).numpy()
        for _ in range(8):  # guard band around the threshold, as in the sweep test
            cur, prev = wl.indicator_pair(w.W, n_el, target, 6000 + s)
            want = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), off, step, w.warmup_m, eps, acc_o)
            margin = np.abs(acc_o + want["l1rel"] - eps)[step >= w.warmup_m]
            if margin.size == 0 or margin.min() > 1e-3 * eps:
                break
            target = target * 1.03
        assert margin.size == 0 or margin.min() > 1e-3 * eps
        got = ctx.chunk_decide(cur.cuda(), prev.cuda(), off, i32(step), w.warmup_m, eps, acc_g)
        torch.cuda.synchronize()
        assert got["recompute"].cpu().numpy().tolist() == want["recompute"].tolist(), f"step {s}"
        assert got["active_ids"].cpu().numpy()[:want["n_active"]].tolist() == want["active_ids"].tolist()
        acc_o = want["acc"]
        active = want["active_ids"].tolist()
        n_forced += int((step < w.warmup_m).sum())
        n_reused += w.W - len(active)
        assert all(c in active for c in range(w.W) if step[c] < w.warmup_m)  # warm-up blocks always compute
        if s in (3, 8, 13):
            O = O0.cuda().clone()
            ctx.chunk_attention(Qg, Kg, Vg, q_off, vis, slo, spo, got["active_ids"], got["n_active"], O)
            torch.cuda.synchronize()
            rows = wl.sample_rows(w, 16, s)
            rows = rows[np.isin(rows // w.n_c, active)]
            if len(rows):
                O_want, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, active,
                                                   sample_rows=rows)
                _check_attention(O.double().cpu().numpy()[:, rows], O_want)
            for c in range(w.W):
                if c not in active:
                    assert torch.equal(O[:, q_off[c]:q_off[c + 1]].cpu(), O0[:, q_off[c]:q_off[c + 1]])
    assert n_forced > 0 and n_reused > 0


# ------------------------------------------------------------------------------------ full-size compression events

def _guarded(H, n_keep, d, dtype):
    """A destination [H, n_keep, d] with one canary row before and one after every head's rows."""
    buf = torch.full((H, n_keep + 2, d), 7.0, dtype=dtype, device="cuda")
    return buf, buf[:, 1:n_keep + 1]


@pytest.mark.parametrize("name", ["cached_step_bf16", "streaming_bf16", "sweep_bf16"])
def test_compression_event_at_full_size_every_element(ctx, name):
    # One compression event of the configuration exactly as the benchmark launches it (all heads, L_k candidates,
    # budget B): the scores against the oracle on every element; the selection on the library's own fp32 scores
    # fed to both sides, indices bit-exact; the compacted K and V rows byte-exact; canary rows before and after
    # every destination head untouched.
    w = wl.CONFIGS[name]
    Q_obs, K, V = wl.candidates(w)
    Kg, Vg = K.cuda(), V.cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    imp = torch.empty((w.H, w.L_k), device="cuda")
    red = torch.empty((w.H, w.L_k), device="cuda")
    got = ctx.kv_score(Q_obs.cuda(), Kg, lambda_=w.lam, pool_k=w.pool_k, imp=imp, red=red, status=status)
    K_buf, K_dst = _guarded(w.H, w.B, w.d, K.dtype)
    V_buf, V_dst = _guarded(w.H, w.B, w.d, K.dtype)
    sel = ctx.kv_select_compact(got["score"], w.B, Kg, Vg, K_dst, V_dst, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    want = oracle.kv_score(wl.bits(Q_obs), wl.bits(K), lambda_=w.lam, pool_k=w.pool_k)
    for nm, g_, w_ in (("imp", imp, want["imp"]), ("red", red, want["red"]),
                       ("score", got["score"], want["score"].astype(np.float64))):
        g_ = g_.double().cpu().numpy()
        assert (np.abs(g_ - w_) <= 1e-4 * np.abs(w_).max(axis=1, keepdims=True)).all(), nm
    score = got["score"].cpu().numpy()
    want_sel = oracle.kv_select_compact(score, w.B, wl.bits(K), wl.bits(V))
    assert int(sel["n_kept"].item()) == want_sel["n_kept"] == w.B
    assert np.array_equal(sel["kept_idx"].cpu().numpy(), want_sel["kept_idx"])
    assert np.array_equal(wl.bits(K_dst.cpu()), want_sel["K_dst"])
    assert np.array_equal(wl.bits(V_dst.cpu()), want_sel["V_dst"])
    for buf in (K_buf, V_buf):
        assert (buf[:, 0] == 7.0).all() and (buf[:, w.B + 1] == 7.0).all()


def test_streaming_generation_at_full_width(ctx):
    # config 4 at full width (24 heads, chunks of 4680 tokens, budget 28080): the history starts full, then eight
    # chunks are generated one after another, each with S denoising steps of attention over [history | itself]
    # (sampled rows) and an accumulated importance, and a real compression 32760 -> 28080 after every chunk,
    # selection bit-exact on the library's scores and rows byte-exact, every time.
    full = wl.CONFIGS["streaming_bf16"]
    H, d, n_c, B, S = full.H, full.d, full.n_c, full.B, full.n_steps
    n_chunks, n_fill = 8, full.B // full.n_c
    keys = list(wl.ar1_keys(H, n_fill + n_chunks, n_c, d, seed=full.seed, sigma=full.sigma))
    hist_K = torch.cat(keys[:n_fill], 1).contiguous()
    hist_V = wl.normal((H, B, d), 6999, full.sigma, torch.bfloat16)
    q_off, vis = np.array([0, n_c], np.int32), np.array([B + n_c], np.int32)
    slo, spo = np.array([0, B, B + n_c], np.int32), np.array([0, B], np.int32)
    shape = wl.Workload("x", "bf16", H=H, d=d, W=1, n_c=n_c, B=0, L_k=0, seed=0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for c in range(n_chunks):
        K_all = torch.cat([hist_K, keys[n_fill + c]], 1).contiguous()
        V_all = torch.cat([hist_V, wl.normal((H, n_c, d), 7000 + c, full.sigma, torch.bfloat16)], 1).contiguous()
        Kg, Vg = K_all.cuda(), V_all.cuda()
        acc_g = torch.zeros((H, B + n_c), device="cuda")
        acc_o = np.zeros((H, B + n_c), np.float64)
        for s in range(S):
            Q = wl.normal((H, n_c, d), 8000 + 10 * c + s, full.sigma, torch.bfloat16)
            O = torch.zeros((H, n_c, d), dtype=torch.bfloat16, device="cuda")
            ctx.chunk_attention(Q.cuda(), Kg, Vg, q_off, vis, slo, spo, i32([0]), i32([1]), O, status=status)
            rows = wl.sample_rows(shape, 8, 10 * c + s)
            O_want, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K_all), wl.bits(V_all), q_off, vis, slo, spo, [0],
                                               sample_rows=rows)
            _check_attention(O[:, torch.as_tensor(rows, dtype=torch.long, device="cuda")].double().cpu().numpy(), O_want)
            Q_obs = Q[:, n_c - full.L_q_obs:].contiguous()
            phase = 2 if s == S - 1 else 1
            want = oracle.kv_score(wl.bits(Q_obs), wl.bits(K_all), lambda_=full.lam, pool_k=full.pool_k,
                                   imp_accum=acc_o, accum_phase=phase, n_steps=S)
            got = ctx.kv_score(Q_obs.cuda(), Kg, lambda_=full.lam, pool_k=full.pool_k, imp_accum=acc_g,
                               accum_phase=phase, n_steps=S, status=status)
        torch.cuda.synchronize()
        score = got["score"].cpu().numpy()
        assert np.abs(score - want["score"]).max() <= 1e-4 * np.abs(want["score"]).max()
        sel = ctx.kv_select_compact(got["score"], B, Kg, Vg, status=status)
        want_sel = oracle.kv_select_compact(score, B, wl.bits(K_all), wl.bits(V_all))
        torch.cuda.synchronize()
        assert status.item() == 0
        assert sel["kept_idx"].shape == (H, B)
        assert np.array_equal(sel["kept_idx"].cpu().numpy(), want_sel["kept_idx"])
        assert np.array_equal(wl.bits(sel["K_dst"].cpu()), want_sel["K_dst"])
        assert np.array_equal(wl.bits(sel["V_dst"].cpu()), want_sel["V_dst"])
        assert not np.array_equal(want_sel["kept_idx"][0], np.arange(B, dtype=np.int32))  # something was dropped
        hist_K, hist_V = sel["K_dst"].cpu(), sel["V_dst"].cpu()


# ------------------------------------------------------------------------------------ the step as a CUDA graph

def test_whole_step_replays_from_a_cuda_graph(ctx):
    # No call allocates, synchronises or leaves its stream, and the work list never returns to the host, so one step
    # (decide -> attention -> score -> select + compact -> cache apply) can be captured into a CUDA graph once and
    # replayed on new data: the replay must give bit for bit what the same calls give when launched one by one, also
    # when the new data changes which chunks are active.
    w = wl.Workload("g", "bf16", H=4, d=128, W=3, n_c=333, B=211, L_k=544, seed=55, sigma=0.5, keys="clustered")
    n_el = w.n_c * w.hidden
    off = np.arange(w.W + 1, dtype=np.int64) * n_el
    q_off, vis, slo, spo = wl.prefix_layout(w)
    dev = "cuda"

    def inputs(seed, targets):
        cur, prev = wl.indicator_pair(w.W, n_el, targets, seed)
        Q, K, V = wl.qkv(w, seed)
        return dict(cur=cur, prev=prev, Q=Q, K=K, V=V)

    first, second = inputs(1, [0.3, 0.01, 0.3]), inputs(2, [0.01, 0.3, 0.3])
    st = {k: v.to(dev).clone() for k, v in first.items()}  # static input buffers of the graph
    out = dict(acc=torch.zeros(w.W, device=dev), l1rel=torch.empty(w.W, device=dev),
               recompute=torch.empty(w.W, dtype=torch.uint8, device=dev),
               active_ids=torch.empty(w.W, dtype=torch.int32, device=dev), n_active=torch.empty(1, dtype=torch.int32, device=dev),
               O=torch.zeros((w.H, w.window_rows, w.d), dtype=torch.bfloat16, device=dev),
               score=torch.empty((w.H, w.L_k), device=dev), kept=torch.empty((w.H, w.B), dtype=torch.int32, device=dev),
               n_kept=torch.empty(1, dtype=torch.int32, device=dev),
               K_dst=torch.empty((w.H, w.B, w.d), dtype=torch.bfloat16, device=dev),
               V_dst=torch.empty((w.H, w.B, w.d), dtype=torch.bfloat16, device=dev),
               y=torch.zeros(w.W * n_el, dtype=torch.bfloat16, device=dev),
               cache=torch.zeros(w.W * n_el, dtype=torch.bfloat16, device=dev),
               status=torch.zeros(1, dtype=torch.int32, device=dev))
    step_no = torch.full((w.W,), 4, dtype=torch.int32, device=dev)

    def step():
        ctx.chunk_decide(st["cur"], st["prev"], off, step_no, 1, 0.1, out["acc"], l1rel=out["l1rel"],
                         recompute=out["recompute"], active_ids=out["active_ids"], n_active=out["n_active"], status=out["status"])
        ctx.chunk_attention(st["Q"], st["K"], st["V"], q_off, vis, slo, spo, out["active_ids"], out["n_active"], out["O"],
                            status=out["status"])
        ctx.kv_score(st["Q"][:, -w.L_q_obs:], st["K"][:, :w.L_k], score=out["score"], status=out["status"])
        ctx.kv_select_compact(out["score"], w.B, st["K"][:, :w.L_k], st["V"][:, :w.L_k], out["K_dst"], out["V_dst"],
                              kept_idx=out["kept"], n_kept=out["n_kept"], status=out["status"])
        ctx.chunk_cache_apply(st["cur"], out["y"], out["cache"], off, out["recompute"], status=out["status"])

    def reset():
        out["acc"].zero_(); out["O"].zero_(); out["y"].zero_(); out["cache"].zero_()

    def snapshot():
        return {k: v.clone() for k, v in out.items()}

    # eager references for both data sets (this also sizes the binding's cached workspaces before the capture)
    want = []
    for data in (first, second):
        for k, v in data.items():
            st[k].copy_(v)
        reset()
        step()
        torch.cuda.synchronize()
        want.append(snapshot())
    assert want[0]["recompute"].cpu().tolist() == [1, 0, 1] and want[1]["recompute"].cpu().tolist() == [0, 1, 1]
    # capture once ...
    for k, v in first.items():
        st[k].copy_(v)
    reset()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    # ... replay on both data sets
    for data, ref in ((first, want[0]), (second, want[1]), (first, want[0])):
        for k, v in data.items():
            st[k].copy_(v)
        reset()
        graph.replay()
        torch.cuda.synchronize()
        for k in out:
            assert torch.equal(out[k].view(torch.uint8) if out[k].dtype == torch.bfloat16 else out[k],
                               ref[k].view(torch.uint8) if ref[k].dtype == torch.bfloat16 else ref[k]), k
    assert out["status"].item() == 0
