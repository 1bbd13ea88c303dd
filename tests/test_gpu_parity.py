"""Parity of the CUDA library (through its C ABI) with the CPU oracle, on the same seeded inputs.

Bars: decisions, active lists and kept indices bit-exact; compacted rows byte-exact; fp32 outputs
within 1e-4; bf16 attention within max-abs 1e-2 and relative-L2 1e-2; importance / redundancy /
score within 1e-4 of the row maximum.
"""
import math

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


def dev(t):
    return t.cuda()


def i32(x):
    return torch.as_tensor(np.asarray(x), dtype=torch.int32).cuda()


# ------------------------------------------------------------------------------------ decide

def _run_decide_sequence(ctx, dtype, lens, n_steps, eps, m, seed, r_hi=0.2):
    n = len(lens)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    acc_o = np.zeros(n, np.float32)
    acc_g = torch.zeros(n, dtype=torch.float32, device="cuda")
    min_margin = math.inf
    for s in range(n_steps):
        target = wl.uniform((n,), seed * 100 + s, 0.0, r_hi)
        parts = [wl.indicator_pair(1, int(L), [float(target[c])], seed * 1000 + s * 10 + c, dtype=dtype)
                 for c, L in enumerate(lens)]
        cur = torch.cat([p[0] for p in parts])
        prev = torch.cat([p[1] for p in parts])
        step = np.full(n, s, np.int32)
        want = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), off, step, m, eps, acc_o)
        margin = np.abs(acc_o + want["l1rel"] - eps)
        min_margin = min(min_margin, float(margin[step >= m].min()) if (step >= m).any() else math.inf)
        got = ctx.chunk_decide(dev(cur), dev(prev), off, i32(step), m, eps, acc_g)
        torch.cuda.synchronize()
        assert got["recompute"].cpu().numpy().tolist() == want["recompute"].tolist(), f"step {s}"
        assert int(got["n_active"].item()) == want["n_active"]
        ids = got["active_ids"].cpu().numpy()
        assert ids[:want["n_active"]].tolist() == want["active_ids"].tolist()
        assert (ids[want["n_active"]:] == -1).all()
        np.testing.assert_allclose(got["l1rel"].cpu().numpy(), want["l1rel"], rtol=2e-6)
        np.testing.assert_allclose(acc_g.cpu().numpy(), want["acc"], rtol=4e-6, atol=1e-9)
        acc_o = want["acc"]
    # the decisions above are only meaningful if no step sat on the threshold
    assert min_margin > 1e-3 * eps, f"a step came within {min_margin} of eps; change the seed"


def test_decide_tiny_f32_config(ctx):
    w = wl.CONFIGS["tiny_f32"]
    _run_decide_sequence(ctx, torch.float32, [w.n_c * w.hidden] * w.W, w.n_steps, w.eps, w.warmup_m, w.seed)


def test_decide_bf16_ragged_and_unaligned(ctx):
    # lengths that are not multiples of the slab, of the vector, or aligned to 16 bytes
    _run_decide_sequence(ctx, torch.bfloat16, [8192 * 3 + 8, 40000, 8, 123456], 4, 0.1, 1, 7)
    _run_decide_sequence(ctx, torch.bfloat16, [1001, 77777, 3], 3, 0.1, 1, 8)
    _run_decide_sequence(ctx, torch.float32, [4099, 65536 + 4, 5], 3, 0.1, 2, 9)


def test_decide_special_cases(ctx):
    n = 4096
    prev = torch.ones(2 * n)
    cur = torch.full((2 * n,), 1.25)
    cur[n:] = 0.0
    prev[n:] = 0.0  # second chunk: zero over zero -> r = 0
    off = [0, n, 2 * n]
    acc = torch.zeros(2, device="cuda")
    out = ctx.chunk_decide(dev(cur), dev(prev), off, i32([3, 3]), 1, 0.25, acc)
    assert out["recompute"].cpu().tolist() == [0, 0]  # s == eps reuses (strict >)
    assert out["l1rel"].cpu().tolist() == [0.25, 0.0]
    cur[n:] = 1.0  # zero denominator, positive numerator -> +inf -> recompute
    acc.zero_()
    out = ctx.chunk_decide(dev(cur), dev(prev), off, i32([3, 3]), 1, 10.0, acc)
    assert out["recompute"].cpu().tolist() == [0, 1] and math.isinf(out["l1rel"][1].item())
    # forced chunk and warm-up reset the accumulator
    acc.fill_(0.2)
    out = ctx.chunk_decide(dev(cur), dev(prev), off, i32([0, 9]), 1, 1e9, acc,
                           force=torch.tensor([0, 1], dtype=torch.uint8).cuda())
    assert out["recompute"].cpu().tolist() == [1, 1] and acc.cpu().tolist() == [0.0, 0.0]
    # run-to-run bit reproducibility
    cur2, prev2 = wl.indicator_pair(3, 100000, [0.1, 0.2, 0.3], 3)
    a = ctx.chunk_decide(dev(cur2), dev(prev2), [0, 100000, 200000, 300000], i32([5] * 3), 1, 0.5,
                         torch.zeros(3, device="cuda"))["l1rel"].clone()
    b = ctx.chunk_decide(dev(cur2), dev(prev2), [0, 100000, 200000, 300000], i32([5] * 3), 1, 0.5,
                         torch.zeros(3, device="cuda"))["l1rel"]
    assert torch.equal(a, b)


@pytest.mark.parametrize("name", ["cached_step_bf16"])
def test_decide_full_size(ctx, name):
    w = wl.CONFIGS[name]
    lens = [w.n_c * w.hidden] * w.W
    _run_decide_sequence(ctx, w.torch_dtype, lens, 2, 0.1, 1, w.seed)


def test_decide_uniform_policy_sequence(ctx):
    # the uniform policy (one shared decision; a re-initialised chunk is computed on its own) over ten steps,
    # ragged chunk lengths, bit-exact flags against the oracle, no step inside the guard band of the threshold
    from paper_2602_10825_b200 import binding
    lens = [40000, 8192 * 3 + 8, 123456, 1001]
    n, eps, m = len(lens), 0.12, 1
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    acc_o = np.zeros(n, np.float32)
    acc_g = torch.zeros(n, device="cuda")
    seen = set()
    for s in range(10):
        target = wl.uniform((n,), 770 + s, 0.0, 0.1)
        parts = [wl.indicator_pair(1, int(L), [float(target[c])], 7700 + s * 10 + c) for c, L in enumerate(lens)]
        cur, prev = torch.cat([p[0] for p in parts]), torch.cat([p[1] for p in parts])
        step = np.full(n, s, np.int32)
        if s >= 4:
            step[2] = s - 4  # chunk 2 is re-initialised at step 4: in warm-up there, sharing again afterwards
        force = np.array([0, 1 if s == 7 else 0, 0, 0], np.uint8)
        want = oracle.chunk_decide_uniform(wl.bits(cur), wl.bits(prev), off, step, m, eps, acc_o, force=force)
        sharing = (step >= m) & (force == 0)
        if sharing.any():
            first = int(np.flatnonzero(sharing)[0])
            assert abs(acc_o[first] + want["l1rel"][first] - eps) > 1e-3 * eps, "inside the guard band: change the seed"
        got = ctx.chunk_decide(dev(cur), dev(prev), off, i32(step), m, eps, acc_g, force=torch.from_numpy(force).cuda(),
                               policy=binding.POLICY_UNIFORM)
        torch.cuda.synchronize()
        assert got["recompute"].cpu().numpy().tolist() == want["recompute"].tolist(), f"step {s}"
        assert int(got["n_active"].item()) == want["n_active"]
        ids = got["active_ids"].cpu().numpy()
        assert ids[:want["n_active"]].tolist() == want["active_ids"].tolist() and (ids[want["n_active"]:] == -1).all()
        np.testing.assert_allclose(got["l1rel"].cpu().numpy(), want["l1rel"], rtol=2e-6)
        np.testing.assert_allclose(acc_g.cpu().numpy(), want["acc"], rtol=4e-6, atol=1e-9)
        acc_o = want["acc"]
        seen.add(tuple(want["recompute"].tolist()))
    assert len(seen) >= 3  # all computed, all reused, and a mixed step around the re-initialised chunk


# ------------------------------------------------------------------------------------ activation cache

@pytest.mark.parametrize("dtype,lens", [(torch.bfloat16, [8192 * 3 + 8, 40000, 8, 123456]),  # 16-byte aligned offsets
                                        (torch.bfloat16, [1001, 77777, 3]),                   # unaligned: scalar path
                                        (torch.float32, [4100, 65536 + 4, 0, 12])])
def test_cache_apply_bit_exact(ctx, dtype, lens):
    # two steps: every chunk computed (the residuals are stored), then a mixed step (skipped chunks are served from
    # the cache, computed ones refresh it); outputs and cache bit for bit against the oracle, untouched parts intact
    n = len(lens)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    E = int(off[-1])
    cache_o = wl.bits(wl.normal((E,), 501, 1.0, dtype))
    cache_g = dev(wl.normal((E,), 501, 1.0, dtype))
    for s, rec in enumerate([[1] * n, [(c + 1) % 2 for c in range(n)], [0] * n]):
        x = wl.normal((E,), 510 + s, 2.0, dtype)
        y = wl.normal((E,), 520 + s, 2.0, dtype)
        y_o, cache_o = oracle.chunk_cache_apply(wl.bits(x), wl.bits(y), cache_o, off, rec)
        y_g = dev(y)
        ctx.chunk_cache_apply(dev(x), y_g, cache_g, off, torch.tensor(rec, dtype=torch.uint8).cuda())
        torch.cuda.synchronize()
        assert np.array_equal(wl.bits(y_g.cpu()), y_o), f"step {s}"
        assert np.array_equal(wl.bits(cache_g.cpu()), cache_o), f"step {s}"


def test_cache_apply_full_size_follows_the_decision_on_the_device(ctx):
    # config 3's indicator tensors (8 chunks x 4680 tokens x 3072): decide, then serve the skipped chunks, the flags
    # going from one call to the other in device memory; every element against the oracle
    w = wl.CONFIGS["cached_step_bf16"]
    n_el = w.n_c * w.hidden
    off = np.arange(w.W + 1, dtype=np.int64) * n_el
    target = [0.3, 0.01, 0.3, 0.02, 0.01, 0.3, 0.02, 0.3]
    cur, prev = wl.indicator_pair(w.W, n_el, target, 4)
    step = np.full(w.W, 6, np.int32)
    want_d = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), off, step, 1, 0.1, np.zeros(w.W, np.float32))
    dec = ctx.chunk_decide(dev(cur), dev(prev), off, i32(step), 1, 0.1, torch.zeros(w.W, device="cuda"))
    y = wl.normal((w.W * n_el,), 44, 1.0, torch.bfloat16)
    cache = wl.normal((w.W * n_el,), 45, 0.1, torch.bfloat16)
    y_g, cache_g = dev(y), dev(cache)
    ctx.chunk_cache_apply(dev(cur), y_g, cache_g, off, dec["recompute"])
    torch.cuda.synchronize()
    assert dec["recompute"].cpu().numpy().tolist() == want_d["recompute"].tolist() == [1, 0, 1, 0, 0, 1, 0, 1]
    y_o, cache_o = oracle.chunk_cache_apply(wl.bits(cur), wl.bits(y), wl.bits(cache), off, want_d["recompute"])
    assert np.array_equal(wl.bits(y_g.cpu()), y_o)
    assert np.array_equal(wl.bits(cache_g.cpu()), cache_o)


# ------------------------------------------------------------------------------------ attention

def _attention_case(ctx, w, active, *, impl=0, token_map=False, sample=None, atol, rel_l2, check_lse=True):
    Q, K, V = wl.qkv(w)
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O0 = wl.normal((w.H, w.window_rows, w.d), 999, 1.0, w.torch_dtype)  # "cached outputs" of earlier steps
    Og = dev(O0).clone()
    lse_g = torch.full((w.H, w.window_rows), float("nan"), device="cuda")
    tok = None
    kw = {}
    if token_map:
        rng = np.random.default_rng(w.seed)
        L = K.shape[1]
        tok = np.stack([rng.permutation(L) for _ in range(w.H)]).astype(np.int32)
        K2, V2 = torch.empty_like(K), torch.empty_like(V)
        for h in range(w.H):
            K2[h, tok[h]] = K[h]
            V2[h, tok[h]] = V[h]
        K, V = K2, V2
        kw["kv_token_index"] = i32(tok)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n_act = i32([len(active)])
    act = i32(list(active) + [-1] * (w.W - len(active)))
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, None if token_map else slo,
                        None if token_map else spo, act, n_act, Og, lse=lse_g, impl=impl, status=status, **kw)
    torch.cuda.synchronize()
    assert status.item() == 0
    O_want, lse_want = oracle.chunk_attention(
        wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, None if token_map else slo,
        None if token_map else spo, active, kv_token_index=tok, sample_rows=sample,
        O_init=None if sample is not None else O0.double().numpy())
    if sample is not None:
        rows = np.asarray(sample)
        is_act = np.isin(rows // w.n_c, list(active))
        pick = torch.as_tensor(rows[is_act], dtype=torch.long, device="cuda")  # gathered on the device: O is large
        got_s, want_s = Og[:, pick].double().cpu().numpy(), O_want[:, is_act]
        lse_got_s, lse_want_s = lse_g[:, pick].double().cpu().numpy(), lse_want[:, is_act]
    else:
        got = Og.double().cpu().numpy()
        lse_got = lse_g.double().cpu().numpy()
        rows_act = np.concatenate([np.arange(q_off[c], q_off[c + 1]) for c in active]) if active else np.array([], int)
        got_s, want_s = got[:, rows_act], O_want[:, rows_act]
        lse_got_s, lse_want_s = lse_got[:, rows_act], lse_want[:, rows_act]
    if got_s.size:
        assert np.abs(got_s - want_s).max() <= atol
        assert np.linalg.norm(got_s - want_s) <= rel_l2 * np.linalg.norm(want_s)
        if check_lse:
            np.testing.assert_allclose(lse_got_s, lse_want_s, atol=2e-3 if w.dtype == "bf16" else 1e-4)
    # rows of chunks that were not recomputed keep their cached values, bit for bit
    inactive = [c for c in range(w.W) if c not in active]
    for c in inactive:
        assert torch.equal(Og[:, q_off[c]:q_off[c + 1]].cpu(), O0[:, q_off[c]:q_off[c + 1]])
        assert torch.isnan(lse_g[:, q_off[c]:q_off[c + 1]]).all()
    return Og


def test_attention_tiny_f32_config_every_element(ctx):
    w = wl.CONFIGS["tiny_f32"]
    _attention_case(ctx, w, [0, 1, 2, 3], atol=1e-4, rel_l2=1e-4)
    _attention_case(ctx, w, [1, 3], atol=1e-4, rel_l2=1e-4)


def test_attention_all_skip_returns_cached_outputs(ctx):
    w = wl.CONFIGS["tiny_f32"]
    _attention_case(ctx, w, [], atol=0, rel_l2=0)


@pytest.mark.parametrize("dtype,d", [("f32", 128), ("bf16", 64), ("bf16", 128)])
def test_attention_simt_ragged(ctx, dtype, d):
    # chunk length 200 = 6 row-tiles of 32 + 8; budget 77 (not a multiple of the key tile)
    w = wl.Workload("r", dtype, H=3, d=d, W=3, n_c=200, B=77, L_k=277, seed=12, sigma=0.7)
    tol = dict(atol=1e-4, rel_l2=1e-4) if dtype == "f32" else dict(atol=1e-2, rel_l2=1e-2)
    _attention_case(ctx, w, [0, 2], impl=1, **tol)


def test_attention_token_index_map(ctx):
    w = wl.Workload("m", "f32", H=2, d=64, W=2, n_c=96, B=50, L_k=146, seed=13)
    _attention_case(ctx, w, [0, 1], token_map=True, atol=1e-4, rel_l2=1e-4)
    wb = wl.Workload("m", "bf16", H=2, d=128, W=2, n_c=96, B=50, L_k=146, seed=14, sigma=0.5)
    _attention_case(ctx, wb, [1], token_map=True, atol=1e-2, rel_l2=1e-2)
    _attention_case(ctx, wb, [0, 1], token_map=True, impl=2, atol=1e-2, rel_l2=1e-2)  # on the tensor cores: gathered rows


@pytest.mark.parametrize("d", [128, 64])
def test_attention_token_index_map_tensor_cores(ctx, d):
    # bf16 through a per-head token map on the tcgen05 kernel: several key tiles with a ragged end, visible lengths that
    # are not multiples of four, grouped query heads (two query heads share a map), every physical row that no token
    # maps to filled with NaN / infinities / 3e38, a chunk that sees nothing and a chunk that sees one token
    H_q, H_kv, L_log, L_phys = 4, 2, 777, 1500
    rng = np.random.default_rng(21)
    tok = np.stack([rng.permutation(L_phys)[:L_log] for _ in range(H_kv)]).astype(np.int32)
    Q = wl.normal((H_q, 600, d), 71, 0.5, torch.bfloat16)
    K = wl.normal((H_kv, L_phys, d), 72, 0.5, torch.bfloat16)
    V = wl.normal((H_kv, L_phys, d), 73, 0.5, torch.bfloat16)
    bad = torch.tensor([float("nan"), float("inf"), -float("inf"), 3e38, -3e38]).to(torch.bfloat16)
    for h in range(H_kv):
        unused = np.setdiff1d(np.arange(L_phys), tok[h])
        K[h, unused] = bad[torch.arange(len(unused)) % 5][:, None]
        V[h, unused] = bad[(torch.arange(len(unused)) + 2) % 5][:, None]
    q_off = np.array([0, 130, 131, 400, 600], np.int32)
    vis = np.array([L_log, 1, 0, 389], np.int32)
    O0 = wl.normal((H_q, 600, d), 74, 1.0, torch.bfloat16)
    Og = dev(O0).clone()
    lse_g = torch.full((H_q, 600), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    active = [0, 1, 2, 3]
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, None, None, i32(active), i32([4]), Og, lse=lse_g,
                        kv_token_index=i32(tok), impl=2, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    O_want, lse_want = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, None, None, active,
                                              kv_token_index=tok, O_init=O0.double().numpy())
    got = Og.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - O_want).max() <= 1e-2
    assert np.linalg.norm(got - O_want) <= 1e-2 * np.linalg.norm(O_want)
    lg = lse_g.double().cpu().numpy()
    fin = np.isfinite(lse_want)
    np.testing.assert_allclose(lg[fin], lse_want[fin], atol=2e-3)
    assert np.array_equal(np.isneginf(lg), np.isneginf(lse_want))
    # an index outside the store is reported, not followed
    tok_bad = tok.copy()
    tok_bad[1, 5] = L_phys + 7
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, None, None, i32(active), i32([4]), Og, kv_token_index=i32(tok_bad),
                        impl=2, status=status)
    torch.cuda.synchronize()
    assert status.item() == 4  # FC_DEV_BAD_INDEX


def test_attention_through_the_kept_index_map_at_full_size(ctx):
    # config 3: instead of compacting the 23400-token history to the 18720 kept tokens and attending over the compact
    # copy, attend over the uncompacted store through the per-head kept-index list (the window chunks follow the
    # history in the same store).  Sampled rows against the oracle, and against the compact-then-attend result.
    w = wl.CONFIGS["cached_step_bf16"]
    H, d, n_hist = w.H, w.d, w.L_k
    rng = np.random.default_rng(8)
    K = wl.clustered_keys(H, n_hist + w.window_rows, d, 9001)
    V = wl.normal((H, n_hist + w.window_rows, d), 9002, w.sigma, torch.bfloat16)
    Q = wl.normal((H, w.window_rows, d), 9003, w.sigma, torch.bfloat16)
    kept = np.stack([np.sort(rng.choice(n_hist, w.B, replace=False)) for _ in range(H)]).astype(np.int32)
    tok = np.concatenate([kept, np.tile(n_hist + np.arange(w.window_rows, dtype=np.int32), (H, 1))], axis=1)
    q_off, vis, _, _ = wl.prefix_layout(w)
    active = [2, 5, 7]
    rows = wl.sample_rows(w, 192, 5, chunks=active)
    Kg, Vg, Qg = dev(K), dev(V), dev(Q)
    O_map = torch.zeros((H, w.window_rows, d), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.chunk_attention(Qg, Kg, Vg, q_off, vis, None, None, i32(active + [-1] * 5), i32([3]), O_map,
                        kv_token_index=i32(tok), impl=2, status=status)
    # the same through a compact copy [kept history | window] and the segment table
    idx = torch.as_tensor(tok, dtype=torch.long, device="cuda")[:, :, None].expand(H, tok.shape[1], d)
    Kc, Vc = torch.gather(Kg, 1, idx), torch.gather(Vg, 1, idx)
    _, _, slo, spo = wl.prefix_layout(w)
    O_cmp = torch.zeros_like(O_map)
    ctx.chunk_attention(Qg, Kc, Vc, q_off, vis, slo, spo, i32(active + [-1] * 5), i32([3]), O_cmp, impl=2, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert (O_map.float() - O_cmp.float()).abs().max().item() <= 2e-3  # same arithmetic, other addressing
    O_want, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, None, None, active,
                                       kv_token_index=tok, sample_rows=rows)
    got = O_map[:, torch.as_tensor(rows, dtype=torch.long, device="cuda")].double().cpu().numpy()
    assert np.abs(got - O_want).max() <= 1e-2
    assert np.linalg.norm(got - O_want) <= 1e-2 * np.linalg.norm(O_want)


@pytest.mark.parametrize("d", [128, 64])
def test_attention_bf16_tensor_core_small(ctx, d, impl=2):
    # several 128-row tiles with ragged tails in both rows and keys, a clean region and a window
    w = wl.Workload("t", "bf16", H=2, d=d, W=3, n_c=328, B=200, L_k=528, seed=15, sigma=0.5)
    _attention_case(ctx, w, [0, 1, 2], impl=impl, atol=1e-2, rel_l2=1e-2)
    _attention_case(ctx, w, [2], impl=impl, atol=1e-2, rel_l2=1e-2)
    w2 = wl.Workload("t2", "bf16", H=3, d=d, W=2, n_c=1000, B=0, L_k=1000, seed=16, sigma=0.5)
    _attention_case(ctx, w2, [0, 1], impl=impl, atol=1e-2, rel_l2=1e-2)


def _attention_custom(ctx, Q, K, V, q_off, vis, slo, spo, active, impl, O0=None):
    H_q, R, d = Q.shape
    O0 = wl.normal((H_q, R, d), 555, 1.0, torch.bfloat16) if O0 is None else O0
    Og = dev(O0).clone()
    lse_g = torch.full((H_q, R), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    W = len(q_off) - 1
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, slo, spo, i32(list(active) + [-1] * (W - len(active))),
                        i32([len(active)]), Og, lse=lse_g, impl=impl, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    O_want, lse_want = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, active,
                                              O_init=O0.double().numpy())
    got = Og.double().cpu().numpy()
    assert np.abs(got - O_want).max() <= 1e-2
    assert np.linalg.norm(got - O_want) <= 1e-2 * max(np.linalg.norm(O_want), 1e-30)
    rows = np.concatenate([np.arange(q_off[c], q_off[c + 1]) for c in active]) if len(active) else np.array([], int)
    lg, lw = lse_g.double().cpu().numpy()[:, rows], lse_want[:, rows]
    finite = np.isfinite(lw)
    np.testing.assert_allclose(lg[finite], lw[finite], atol=2e-3)
    assert np.array_equal(np.isneginf(lg), np.isneginf(lw))
    return Og


def test_attention_tensor_core_edge_cases(ctx, impl=2):
    d = 128
    # grouped query heads: 4 query heads on 2 key heads
    Q = wl.normal((4, 300, d), 61, 0.5, torch.bfloat16)
    K = wl.normal((2, 400, d), 62, 0.5, torch.bfloat16)
    V = wl.normal((2, 400, d), 63, 0.5, torch.bfloat16)
    q_off, vis = np.array([0, 100, 300], np.int32), np.array([200, 400], np.int32)
    _attention_custom(ctx, Q, K, V, q_off, vis, np.array([0, 400], np.int32), np.array([0], np.int32), [0, 1], impl)
    # a clean region scattered over ten physical segments in shuffled order, chunks of unequal length, one of
    # them empty, visible lengths that are not monotone, a chunk that sees nothing (output 0, LSE -inf)
    rng = np.random.default_rng(3)
    seg_len = [37, 128, 1, 255, 64, 129, 90, 7, 300, 13]
    order = rng.permutation(len(seg_len))
    phys = np.zeros(len(seg_len), np.int64)
    pos = 5
    for s_ in order:  # lay the segments out in shuffled order with gaps between them
        phys[s_] = pos
        pos += seg_len[s_] + int(rng.integers(0, 9))
    slo = np.concatenate([[0], np.cumsum(seg_len)]).astype(np.int32)
    L_phys = pos + 3
    Q = wl.normal((2, 700, d), 64, 0.5, torch.bfloat16)
    K = wl.normal((2, L_phys, d), 65, 0.5, torch.bfloat16)
    V = wl.normal((2, L_phys, d), 66, 0.5, torch.bfloat16)
    q_off = np.array([0, 130, 130, 400, 401, 700], np.int32)  # chunk 1 is empty, chunk 3 has one row
    vis = np.array([slo[-1], 50, 0, 700, 166], np.int32)
    _attention_custom(ctx, Q, K, V, q_off, vis, slo, phys.astype(np.int32), [0, 1, 2, 3, 4], impl)
    _attention_custom(ctx, Q, K, V, q_off, vis, slo, phys.astype(np.int32), [2, 3], impl)
    # nothing active: nothing is written
    O0 = wl.normal((2, 700, d), 67, 1.0, torch.bfloat16)
    Og = _attention_custom(ctx, Q, K, V, q_off, vis, slo, phys.astype(np.int32), [], impl, O0=O0)
    assert torch.equal(Og.cpu(), O0)


@pytest.mark.parametrize("seed", range(8))
def test_attention_tensor_core_random_geometries(ctx, seed, impl=2):
    # Seeded random layouts: head counts and grouping, head dimension, chunks of unequal (also zero) length, a logical
    # key sequence cut into segments of random length laid out in shuffled physical order with gaps, visible lengths
    # anywhere between nothing and everything, a random set of active chunks in random order.
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    H_kv, group = int(rng.integers(1, 4)), int(rng.choice([1, 2]))
    W = int(rng.integers(1, 7))
    lens = rng.integers(0, 420, W)
    lens[rng.integers(0, W)] += 1  # at least one row somewhere
    q_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    n_seg = int(rng.integers(1, 9))
    seg_len = rng.integers(1, 300, n_seg)
    slo = np.concatenate([[0], np.cumsum(seg_len)]).astype(np.int32)
    phys, pos = np.zeros(n_seg, np.int32), int(rng.integers(0, 6))
    for s_ in rng.permutation(n_seg):
        phys[s_] = pos
        pos += int(seg_len[s_]) + int(rng.integers(0, 40))
    L_phys = pos + int(rng.integers(0, 5))
    vis = rng.integers(0, slo[-1] + 1, W).astype(np.int32)
    vis[rng.integers(0, W)] = slo[-1]
    active = [int(c) for c in rng.permutation(W)[:int(rng.integers(1, W + 1))]]
    Q = wl.normal((H_kv * group, int(q_off[-1]), d), 7000 + seed, 0.5, torch.bfloat16)
    K = wl.normal((H_kv, L_phys, d), 7100 + seed, 0.5, torch.bfloat16)
    V = wl.normal((H_kv, L_phys, d), 7200 + seed, 0.5, torch.bfloat16)
    _poison_unreferenced_rows(K, V, int(vis.max()), slo, phys)
    Og = _attention_custom(ctx, Q, K, V, q_off, vis, slo, phys, active, impl)
    assert torch.isfinite(Og.float()).all()


def _poison_unreferenced_rows(K, V, vis_max, slo, spo):
    """Overwrite every physical K/V row that no visible logical token maps to with NaN, +-inf and +-3e38."""
    L = K.shape[1]
    used = np.zeros(L, bool)
    for s_ in range(len(spo)):
        n = min(int(slo[s_ + 1]), vis_max) - int(slo[s_])
        if n > 0:
            used[int(spo[s_]):int(spo[s_]) + n] = True
    bad = torch.tensor([float("nan"), float("inf"), -float("inf"), 3e38, -3e38], dtype=torch.float32)
    rows = np.flatnonzero(~used)
    fill = bad[torch.arange(len(rows)) % 5].to(torch.bfloat16)[None, :, None]
    K[:, rows] = fill
    V[:, rows] = fill.flip(1)
    return len(rows)


@pytest.mark.parametrize("d", [128, 64])
def test_attention_ignores_rows_outside_the_visible_segments(ctx, d, impl=2):
    # The K/V buffer of the method has slots that are not written yet, and a segment's last 128-row tile drags in
    # whatever follows the segment.  Every such row is filled with NaN, infinities and 3e38 here: the outputs must
    # still match the oracle (which never reads those rows) and be finite.
    rng = np.random.default_rng(4)
    # (1) a clean region scattered over segments with gaps, as in the edge-case test
    seg_len = [37, 128, 1, 255, 64, 129, 90, 7, 300, 13]
    order = rng.permutation(len(seg_len))
    phys = np.zeros(len(seg_len), np.int64)
    pos = 5
    for s_ in order:
        phys[s_] = pos
        pos += seg_len[s_] + int(rng.integers(1, 9))
    slo = np.concatenate([[0], np.cumsum(seg_len)]).astype(np.int32)
    L_phys = pos + 130
    Q = wl.normal((2, 700, d), 64, 0.5, torch.bfloat16)
    K = wl.normal((2, L_phys, d), 65, 0.5, torch.bfloat16)
    V = wl.normal((2, L_phys, d), 66, 0.5, torch.bfloat16)
    q_off = np.array([0, 130, 400, 700], np.int32)
    vis = np.array([slo[-1], 700, 166], np.int32)
    assert _poison_unreferenced_rows(K, V, int(slo[-1]), slo, phys) > 100
    Og = _attention_custom(ctx, Q, K, V, q_off, vis, slo, phys.astype(np.int32), [0, 1, 2], impl)
    assert torch.isfinite(Og.float()).all()
    # (2) the prefix layout [clean region | gap | chunk 0 | gap | chunk 1 | unwritten rest], the second chunk's slot
    # only partly written: chunk 1 sees 100 of its 328 rows, the other 228 are poison inside its own segment
    B, n_c = 200, 328
    spo = np.array([0, B + 56, B + 56 + n_c + 100], np.int32)
    slo = np.array([0, B, B + n_c, B + 2 * n_c], np.int32)
    L_phys = int(spo[2]) + n_c + 77
    Q = wl.normal((3, 2 * n_c, d), 67, 0.5, torch.bfloat16)
    K = wl.normal((3, L_phys, d), 68, 0.5, torch.bfloat16)
    V = wl.normal((3, L_phys, d), 69, 0.5, torch.bfloat16)
    q_off = np.array([0, n_c, 2 * n_c], np.int32)
    vis = np.array([B + n_c, B + n_c + 100], np.int32)
    assert _poison_unreferenced_rows(K, V, int(vis[1]), slo, spo) > 400
    Og = _attention_custom(ctx, Q, K, V, q_off, vis, slo, spo, [0, 1], impl)
    assert torch.isfinite(Og.float()).all()
    # the CUDA-core kernel reads through the same tables
    Og = _attention_custom(ctx, Q, K, V, q_off, vis, slo, spo, [0, 1], 1)
    assert torch.isfinite(Og.float()).all()


def test_attention_bf16_many_items_per_cta(ctx, impl=2):
    # more work items than SMs, of very different lengths: exercises the device-side item queue
    w = wl.Workload("q", "bf16", H=40, d=128, W=6, n_c=520, B=300, L_k=820, seed=18, sigma=0.5)
    _attention_case(ctx, w, [0, 1, 3, 5], impl=impl, sample=wl.sample_rows(w, 40, 1), atol=1e-2, rel_l2=1e-2)


# The launch configurations the benchmark times, at full size, on sampled query rows over the full key range:
# boundary rows of every active chunk plus uniform draws from the active chunks (4096 distinct rows on each of the
# four full-size configurations; the extra cases, a sparse sweep list and the second model family, take 1024).
FULL_SIZE_CASES = [
    ("single_step_bf16", [0, 1, 2, 3], 4096),
    ("cached_step_bf16", [2, 5, 7], 4096),
    ("streaming_bf16", [0], 4096),                 # one chunk over the 28080-token history
    ("sweep_bf16", list(range(16)), 4096),         # every chunk of the window recomputed
    ("sweep_bf16", [1, 4, 9, 15], 1024),           # a sparse active list late in the sweep
    ("skyreels_bf16", [0, 2, 3], 1024),
]


@pytest.mark.parametrize("name,active,n_uniform", FULL_SIZE_CASES,
                         ids=[f"{n}-{len(a)}of{wl.CONFIGS[n].W}" for n, a, _ in FULL_SIZE_CASES])
def test_attention_full_size_sampled_rows(ctx, name, active, n_uniform):
    w = wl.CONFIGS[name]
    rows = wl.sample_rows(w, n_uniform, 2, chunks=active)
    assert len(rows) >= n_uniform * 0.9
    _attention_case(ctx, w, active, sample=rows, atol=1e-2, rel_l2=1e-2)
    torch.cuda.empty_cache()


def test_attention_bf16_mid_size_every_element(ctx):
    # every output element of a case with dozens of work items per head: 10 query tiles per chunk with a ragged
    # last one, up to 52 key tiles per item, a clean region that ends inside a key tile
    w = wl.Workload("mid", "bf16", H=4, d=128, W=4, n_c=1160, B=2000, L_k=3160, seed=18, sigma=0.5)
    _attention_case(ctx, w, [0, 1, 2, 3], impl=2, atol=1e-2, rel_l2=1e-2)
    _attention_case(ctx, w, [3, 1], impl=2, atol=1e-2, rel_l2=1e-2)


def test_attention_bf16_matches_cuda_core_kernel(ctx):
    # second opinion on the device: tensor-core and CUDA-core kernels agree on a mid-size case
    w = wl.Workload("x", "bf16", H=4, d=128, W=4, n_c=1160, B=2000, L_k=3160, seed=17, sigma=0.5)
    a = _attention_case(ctx, w, [0, 2, 3], impl=0, sample=wl.sample_rows(w, 24, 0), atol=1e-2, rel_l2=1e-2)
    b = _attention_case(ctx, w, [0, 2, 3], impl=1, sample=wl.sample_rows(w, 24, 0), atol=1e-2, rel_l2=1e-2)
    assert (a.float() - b.float()).abs().max().item() <= 1e-2


# ------------------------------------------------------------------------------------ scores

def _score_case(ctx, Q, K, lam, pool_k, impl=0):
    want = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=lam, pool_k=pool_k)
    H, L = K.shape[0], K.shape[1]
    imp = torch.empty((H, L), device="cuda")
    red = torch.empty((H, L), device="cuda")
    got = ctx.kv_score(dev(Q), dev(K), lambda_=lam, pool_k=pool_k, imp=imp, red=red, impl=impl)
    torch.cuda.synchronize()
    for name, g, wnt in (("imp", imp, want["imp"]), ("red", red, want["red"]),
                         ("score", got["score"], want["score"].astype(np.float64))):
        g = g.double().cpu().numpy()
        bound = 1e-4 * np.abs(wnt).max(axis=1, keepdims=True)
        assert (np.abs(g - wnt) <= bound).all(), name
    return got["score"], want["score"]


def test_score_tiny_f32_config(ctx):
    w = wl.CONFIGS["tiny_f32"]
    Q_obs, K, _ = wl.candidates(w)
    _score_case(ctx, Q_obs, K, w.lam, w.pool_k)


@pytest.mark.parametrize("impl", [1, 2])  # CUDA-core and tensor-core pipelines
@pytest.mark.parametrize("keys", ["normal", "clustered"])
def test_score_bf16_ragged(ctx, keys, impl):
    w = wl.Workload("s", "bf16", H=3, d=128, W=1, n_c=100, B=1000, L_k=1331, seed=21, sigma=0.5, keys=keys)
    Q_obs, K, _ = wl.candidates(w)
    _score_case(ctx, Q_obs, K, 0.07, 7, impl=impl)
    _score_case(ctx, Q_obs, K, 0.5, 1, impl=impl)


@pytest.mark.parametrize("d,L_q,L_k", [(64, 50, 777), (128, 62, 128), (128, 1, 5000), (128, 33, 9000)])
def test_score_tensor_core_shapes(ctx, d, L_q, L_k):
    # d = 64; exactly one tile; a single query; many tiles per slice with a ragged tail
    Q = wl.normal((2, L_q, d), 51, 0.7, torch.bfloat16)
    K = wl.normal((2, L_k, d), 52, 0.7, torch.bfloat16)
    K[1, 5] = 0  # a zero key: its normalised form is 0
    _score_case(ctx, Q, K, 0.07, 7, impl=2)


def test_score_tensor_core_matches_cuda_core_full_size(ctx):
    # config 3's compression event: both pipelines on every element
    w = wl.CONFIGS["cached_step_bf16"]
    Q_obs, K, _ = wl.candidates(w)
    a = ctx.kv_score(dev(Q_obs), dev(K), lambda_=w.lam, pool_k=w.pool_k, impl=1)["score"]
    b = ctx.kv_score(dev(Q_obs), dev(K), lambda_=w.lam, pool_k=w.pool_k, impl=2)["score"]
    torch.cuda.synchronize()
    assert (a - b).abs().max().item() <= 1e-4 * a.abs().max().item()
    want = oracle.kv_score(wl.bits(Q_obs), wl.bits(K), lambda_=w.lam, pool_k=w.pool_k)["score"]
    assert np.abs(b.double().cpu().numpy() - want).max() <= 1e-4 * np.abs(want).max()


@pytest.mark.parametrize("d,L_q,L_k", [(128, 300, 1000), (64, 129, 700), (128, 1560, 2345)])
def test_score_frame_level_queries(ctx, d, L_q, L_k):
    # frame-level query granularity: more observation queries than the token-level pipelines take (two full
    # query tiles and a ragged one; one query past a tile; a whole latent frame), ragged key tiles, a zero key
    Q = wl.normal((2, L_q, d), 61, 0.7, torch.bfloat16)
    K = wl.normal((2, L_k, d), 62, 0.7, torch.bfloat16)
    K[1, 5] = 0
    _score_case(ctx, Q, K, 0.07, 7)


def test_score_frame_level_full_size_two_heads(ctx):
    # one latent frame of queries (1560 rows) against the 24960 candidates of config 2, two heads (the oracle's
    # cost grows with the head count; the kernels' work per head does not depend on it)
    w = wl.CONFIGS["single_step_bf16"]
    Q = wl.normal((2, 1560, w.d), 81, w.sigma, torch.bfloat16)
    K = wl.normal((2, w.L_k, w.d), 82, w.sigma, torch.bfloat16)
    _score_case(ctx, Q, K, w.lam, w.pool_k)


def test_score_frame_level_accumulated_over_steps(ctx):
    K = wl.normal((2, 900, 128), 71, 0.5, torch.bfloat16)
    Qs = [wl.normal((2, 200, 128), 72 + s, 0.5, torch.bfloat16) for s in range(2)]
    acc_o = np.zeros((2, 900), np.float64)
    acc_g = torch.zeros((2, 900), device="cuda")
    for s, q in enumerate(Qs):
        phase = 2 if s == 1 else 1
        want = oracle.kv_score(wl.bits(q), wl.bits(K), imp_accum=acc_o, accum_phase=phase, n_steps=2)
        imp = torch.empty((2, 900), device="cuda")
        got = ctx.kv_score(dev(q), dev(K), imp_accum=acc_g, accum_phase=phase, n_steps=2, imp=imp)
    torch.cuda.synchronize()
    np.testing.assert_allclose(imp.cpu().numpy(), want["imp"], rtol=0, atol=1e-4 * want["imp"].max())
    np.testing.assert_allclose(got["score"].cpu().numpy(), want["score"], rtol=0,
                               atol=1e-4 * np.abs(want["score"]).max())


# Redundancy from explicit similarity tiles (Eq. 11 as written) and the column-maximum variant

@pytest.mark.parametrize("d,L_k,keys", [(128, 1331, "clustered"), (64, 700, "normal"), (128, 4096, "normal"), (128, 130, "normal")])
def test_score_tiled_redundancy_every_element(ctx, d, L_k, keys):
    from paper_2602_10825_b200 import binding
    w = wl.Workload("t", "bf16", H=2, d=d, W=1, n_c=100, B=L_k, L_k=L_k, seed=23, sigma=0.5, keys=keys)
    Q, K, _ = wl.candidates(w)
    K[1, 5] = 0  # a zero key: similarity 0 to everything
    K[0, 9] = K[0, 2]  # an exact duplicate: similarity 1, and the diagonal must still be left out
    for mode_g, mode_o in ((binding.RED_TILED, oracle.RED_PLAIN), (binding.RED_TILED_MAX, oracle.RED_MAXSIM)):
        want = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=0.07, pool_k=7, red_mode=mode_o)
        red = torch.empty((2, L_k), device="cuda")
        imp = torch.empty((2, L_k), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        got = ctx.kv_score(dev(Q), dev(K), lambda_=0.07, pool_k=7, red=red, imp=imp, red_mode=mode_g, status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        for name, g_, w_ in (("imp", imp, want["imp"]), ("red", red, want["red"]),
                             ("score", got["score"], want["score"].astype(np.float64))):
            g_ = g_.double().cpu().numpy()
            assert (np.abs(g_ - w_) <= 1e-4 * np.abs(w_).max(axis=1, keepdims=True)).all(), (name, mode_g)
    # the plain definition and the mean-key identity are the same function: both device modes agree as well
    a = ctx.kv_score(dev(Q), dev(K), red_mode=binding.RED_TILED)["score"]
    b = ctx.kv_score(dev(Q), dev(K), red_mode=binding.RED_MEANKEY)["score"]
    assert (a - b).abs().max().item() <= 1e-4 * b.abs().max().item()


def test_score_tiled_redundancy_full_size(ctx):
    # config 3's compression event (24 heads x 23400 clustered keys) through the dense tiles: Red on every element
    # against the oracle (which uses the mean-key identity at this size), and the softmax arguments of sampled
    # columns against the plain definition evaluated column by column, for the mean and for the maximum
    from paper_2602_10825_b200 import binding
    w = wl.CONFIGS["cached_step_bf16"]
    Q, K, _ = wl.candidates(w)
    Kg, Qg = dev(K), dev(Q)
    want = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=w.lam, pool_k=w.pool_k)
    cols = np.unique(np.concatenate([[0, 1, 127, 128, w.L_k - 1], np.random.default_rng(3).integers(0, w.L_k, 40)])).astype(np.int32)
    for mode_g, mode_o in ((binding.RED_TILED, oracle.RED_PLAIN), (binding.RED_TILED_MAX, oracle.RED_MAXSIM)):
        red = torch.empty((w.H, w.L_k), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        got = ctx.kv_score(Qg, Kg, lambda_=w.lam, pool_k=w.pool_k, red=red, red_mode=mode_g, status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        r = red.double().cpu().numpy()
        assert abs(r.sum(axis=1) - 1).max() < 1e-4
        if mode_g == binding.RED_TILED:
            assert (np.abs(r - want["red"]) <= 1e-4 * want["red"].max(axis=1, keepdims=True)).all()
            assert np.abs(got["score"].double().cpu().numpy() - want["score"]).max() <= 1e-4 * np.abs(want["score"]).max()
        # Red = softmax(a): differences of log Red between columns are differences of a
        a = oracle.key_similarity_columns(wl.bits(K), cols, mode_o)
        d_gpu = np.log(r[:, cols]) - np.log(r[:, cols[:1]])
        d_orc = a - a[:, :1]
        assert np.abs(d_gpu - d_orc).max() <= 1e-4, mode_g


def test_score_gqa_and_d64(ctx):
    Q = wl.normal((4, 20, 64), 31, 1.0)
    K = wl.normal((2, 300, 64), 32, 1.0)
    _score_case(ctx, Q, K, 0.2, 3)


@pytest.mark.parametrize("g,L_q,L_k", [(2, 25, 1331), (4, 50, 2345), (8, 50, 900)])
def test_score_grouped_query_heads_on_tensor_cores(ctx, g, L_q, L_k):
    # grouped query heads, bf16: g heads x L_q rows per key head are g * L_q observation queries of that key head
    # (50 -> the token-level tensor-core passes, 200 and 400 -> the frame-level ones); the importance is the mean over
    # the group's heads and rows
    H_kv = 2
    Q = wl.normal((H_kv * g, L_q, 128), 91, 0.7, torch.bfloat16)
    K = wl.normal((H_kv, L_k, 128), 92, 0.7, torch.bfloat16)
    _score_case(ctx, Q, K, 0.07, 7)
    # the same heads with a gap between them in memory are not one block of rows: the CUDA-core pipeline takes them
    if g * L_q <= 128:
        Qp = torch.zeros((H_kv * g, L_q + 3, 128), dtype=torch.bfloat16)
        Qp[:, :L_q] = Q
        want = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=0.07, pool_k=7)
        got = ctx.kv_score(dev(Qp)[:, :L_q], dev(K), lambda_=0.07, pool_k=7)["score"].double().cpu().numpy()
        assert np.abs(got - want["score"]).max() <= 1e-4 * np.abs(want["score"]).max()


def test_score_accumulated_over_steps(ctx):
    K = wl.normal((2, 700, 128), 41, 0.5, torch.bfloat16)
    Qs = [wl.normal((2, 50, 128), 42 + s, 0.5, torch.bfloat16) for s in range(3)]
    acc_o = np.zeros((2, 700), np.float64)
    acc_g = torch.zeros((2, 700), device="cuda")
    for s, q in enumerate(Qs):
        phase = 2 if s == 2 else 1
        want = oracle.kv_score(wl.bits(q), wl.bits(K), imp_accum=acc_o, accum_phase=phase, n_steps=3)
        imp = torch.empty((2, 700), device="cuda")
        got = ctx.kv_score(dev(q), dev(K), imp_accum=acc_g, accum_phase=phase, n_steps=3, imp=imp)
    torch.cuda.synchronize()
    np.testing.assert_allclose(imp.cpu().numpy(), want["imp"], rtol=0, atol=1e-4 * want["imp"].max())
    np.testing.assert_allclose(got["score"].cpu().numpy(), want["score"], rtol=0,
                               atol=1e-4 * np.abs(want["score"]).max())


def test_attention_logit_jump_far_above_the_running_maximum(ctx):
    # Keys late in the prefix whose logits exceed everything before them by hundreds of log2 units, for single query
    # rows only (the other rows of the warp see nothing unusual): the reference maximum must move for exactly those
    # rows and O be rescaled, whichever unit takes the exponential of that column (columns 6 and 7 of a 64-column
    # half go to the fma pipe, columns 0 and 64 to the special-function unit).
    w = wl.Workload("jump", "bf16", H=2, d=128, W=1, n_c=256, B=1536, L_k=0, seed=91, sigma=0.5)
    Q, K, V = wl.qkv(w)
    Q[:, :, 120:] = 0
    K[:, :, 120:] = 0
    for n, (pos, row) in enumerate(((128 * 5 + 6, 0), (128 * 7 + 71, 37), (128 * 9 + 64, 130), (128 * 11 + 7, 255))):
        Q[:, row, 120 + n] = 8.0           # only this row has a component along axis 120 + n ...
        K[:, pos, 120 + n] = 200.0 * (n + 1)  # ... and only this key: logit 1600 (n+1) / sqrt(128) = 141 (n+1) nats
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O = torch.zeros_like(Q).cuda()
    lse = torch.empty((w.H, w.n_c), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, slo, spo, i32([0]), i32([1]), O, lse=lse, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    O_want, lse_want = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0])
    got = O.double().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - O_want).max() <= 1e-2
    assert np.linalg.norm(got - O_want) <= 1e-2 * np.linalg.norm(O_want)
    np.testing.assert_allclose(lse.double().cpu().numpy(), lse_want, rtol=1e-5, atol=2e-3)
    # the four rows attend to their own key alone
    for pos, row in ((128 * 5 + 6, 0), (128 * 7 + 71, 37), (128 * 9 + 64, 130), (128 * 11 + 7, 255)):
        assert np.abs(got[:, row] - V[:, pos].double().numpy()).max() <= 1e-2


# ------------------------------------------------------------------------------------ select + compact

def _select_case(ctx, score, B, K=None, V=None):
    want = oracle.kv_select_compact(score, B, None if K is None else wl.bits(K), None if V is None else wl.bits(V))
    H, L = score.shape
    n_keep = min(B, L)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if K is not None:
        # canaries around the destination: one extra row per head must stay untouched
        Kd = torch.full((H, n_keep + 1, K.shape[2]), 7.0, dtype=K.dtype, device="cuda")
        Vd = torch.full((H, n_keep + 1, K.shape[2]), 7.0, dtype=K.dtype, device="cuda")
        got = ctx.kv_select_compact(torch.from_numpy(score).cuda(), B, dev(K), dev(V), Kd[:, :n_keep], Vd[:, :n_keep],
                                    status=status)
    else:
        got = ctx.kv_select_compact(torch.from_numpy(score).cuda(), B, status=status)
    torch.cuda.synchronize()
    assert np.array_equal(got["kept_idx"].cpu().numpy(), want["kept_idx"])
    assert int(got["n_kept"].item()) == want["n_kept"] == n_keep
    if K is not None:
        assert np.array_equal(wl.bits(Kd[:, :n_keep].cpu()), want["K_dst"])
        assert np.array_equal(wl.bits(Vd[:, :n_keep].cpu()), want["V_dst"])
        assert (Kd[:, n_keep] == 7.0).all() and (Vd[:, n_keep] == 7.0).all()
    return status.item()


def test_select_bit_exact_with_ties_nan_and_zeros(ctx):
    rng = np.random.default_rng(5)
    score = rng.normal(size=(4, 5000)).astype(np.float32)
    score[:, ::5] = score[:, 2:3]          # one value repeated 1000 times per head
    score[1, 17] = np.nan
    score[2, 100:200] = 0.0
    score[2, 150] = -0.0
    score[3] = 1.0                          # a head where every score ties
    for B in (1, 2, 999, 1000, 1001, 2500, 4999, 5000, 6000):
        st = _select_case(ctx, score, B)
        assert st & 2  # the NaN was reported
    assert _select_case(ctx, np.ascontiguousarray(score[2:]), 700) == 0


def test_select_compact_tiny_and_ragged(ctx):
    w = wl.CONFIGS["tiny_f32"]
    _, K, V = wl.candidates(w)
    score = oracle.kv_score(wl.bits(wl.candidates(w)[0]), wl.bits(K))["score"]
    _select_case(ctx, score, w.B, K, V)
    _select_case(ctx, score, w.L_k, K, V)       # budget = cache length: identity
    _select_case(ctx, score, w.L_k + 100, K, V)  # budget beyond it: identity
    wb = wl.Workload("c", "bf16", H=5, d=128, W=1, n_c=10, B=3001, L_k=4099, seed=6, sigma=0.5)
    _, Kb, Vb = wl.candidates(wb)
    sb = np.random.default_rng(9).normal(size=(5, 4099)).astype(np.float32)
    _select_case(ctx, sb, wb.B, Kb, Vb)
    wc = wl.Workload("c", "bf16", H=2, d=64, W=1, n_c=10, B=100, L_k=333, seed=6, sigma=0.5)
    _, Kc, Vc = wl.candidates(wc)
    _select_case(ctx, sb[:2, :333].copy(), 100, Kc, Vc)


@pytest.mark.parametrize("seed", range(6))
def test_select_random_sizes_and_value_distributions(ctx, seed):
    # Seeded random cases: lengths that do not divide by the cluster size or the vector width, budgets anywhere in
    # [1, L], and score distributions that stress the radix passes: values quantised to a few levels (many ties, tie
    # order decides), a range so narrow that all keys share their leading bits, a mix of signs, denormals and huge
    # values, an already sorted head.
    rng = np.random.default_rng(500 + seed)
    H = int(rng.integers(1, 7))
    L = int(rng.choice([1, 2, 31, 1023, 1025, 4097, 10007, 43681]))
    kind = seed % 6
    if kind == 0:
        score = rng.integers(0, 4, size=(H, L)).astype(np.float32)
    elif kind == 1:
        score = (1.0 + rng.integers(0, 2000, size=(H, L)) * 2.0 ** -23).astype(np.float32)
    elif kind == 2:
        score = (rng.normal(size=(H, L)) * 10.0 ** rng.integers(-42, 38, size=(H, L)).astype(np.float64)).astype(np.float32)
    elif kind == 3:
        score = np.sort(rng.normal(size=(H, L)).astype(np.float32), axis=1)
    elif kind == 4:
        score = -np.abs(rng.normal(size=(H, L))).astype(np.float32)
        score[:, ::7] = -0.0
    else:
        score = rng.random(size=(H, L)).astype(np.float32)
    for B in sorted({1, max(1, L // 3), max(1, L - 1), L, int(rng.integers(1, L + 1))}):
        assert _select_case(ctx, score, B) == 0


def test_select_large_head_falls_back_to_global_keys(ctx):
    rng = np.random.default_rng(11)
    score = rng.normal(size=(2, 70001)).astype(np.float32)  # a cluster of four blocks per head, 70 KB of keys each
    score[:, ::3] = 0.5
    _select_case(ctx, score, 33333)
    # 80 heads leave one block per head, and 60000 keys (240 KB) do not fit its shared memory: the keys are
    # recomputed from the scores in global memory on every pass
    score = rng.normal(size=(80, 60000)).astype(np.float32)
    score[:, ::4] = -0.25
    _select_case(ctx, score, 41234)


def _select_units_case(ctx, score, B, unit, n_protect, K=None, V=None):
    want = oracle.kv_select_units(score, B, unit=unit, n_protect=n_protect)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = ctx.kv_select_compact(torch.from_numpy(score).cuda(), B, None if K is None else dev(K),
                                None if V is None else dev(V), status=status, unit=unit, n_protect=n_protect)
    torch.cuda.synchronize()
    kept = got["kept_idx"].cpu().numpy()
    assert np.array_equal(kept, want["kept_idx"]), (B, unit, n_protect)
    assert int(got["n_kept"].item()) == want["n_kept"]
    if K is not None:  # the rows of the kept tokens, byte for byte
        idx = torch.from_numpy(kept.astype(np.int64))[:, :, None].expand(-1, -1, K.shape[2])
        assert np.array_equal(wl.bits(got["K_dst"].cpu()), wl.bits(torch.gather(K, 1, idx)))
        assert np.array_equal(wl.bits(got["V_dst"].cpu()), wl.bits(torch.gather(V, 1, idx)))
    return status.item()


def test_select_by_units_and_with_a_protected_tail(ctx):
    rng = np.random.default_rng(23)
    score = rng.normal(size=(4, 4800)).astype(np.float32)
    score[:, ::5] = score[:, 2:3]      # many equal scores
    score[1, 17] = np.nan
    score[3] = 1.0                      # a head where everything ties
    # token level with the newest tokens protected (also more protected tokens than the budget holds)
    for B, n_protect in ((1000, 1), (1000, 300), (2500, 2500), (64, 500), (4800, 10)):
        st = _select_units_case(ctx, score, B, 1, n_protect)
        assert st & 2 or B >= 4800  # the NaN was reported (the identity path reports it too)
    # units of 8, 100 and 1600 tokens (a NaN makes its whole unit rank last), with and without protection
    for unit, B, n_protect in ((8, 2400, 0), (8, 2400, 20), (100, 1200, 0), (100, 4800, 0), (1600, 3200, 1), (1600, 1600, 0)):
        _select_units_case(ctx, score, B, unit, n_protect)
    import paper_2602_10825_b200 as fc
    with pytest.raises(fc.FcError, match="invalid"):   # whole units only
        ctx.kv_select_compact(torch.from_numpy(score).cuda(), 1000, unit=7)


@pytest.mark.parametrize("name", ["cached_step_bf16", "sweep_bf16"])
def test_select_by_latent_frames_at_full_size(ctx, name):
    # the key-granularity ablation at the benchmark's sizes: units of one latent frame (30 x 52 = 1560 tokens), scores
    # from the library itself fed to both sides, kept frames bit-exact, compacted rows byte-exact
    w = wl.CONFIGS[name]
    Q_obs, K, V = wl.candidates(w)
    score = ctx.kv_score(dev(Q_obs), dev(K), lambda_=w.lam, pool_k=w.pool_k)["score"].cpu().numpy()
    assert w.L_k % 1560 == 0 and w.B % 1560 == 0
    _select_units_case(ctx, score, w.B, 1560, 0, K, V)
    _select_units_case(ctx, score, w.B, 1560, 1560, K, V)   # the newest frame protected


def test_pipeline_gpu_scores_feed_gpu_select(ctx):
    # end to end on the device: score -> select on the library's own fp32 scores; the oracle's
    # selection on those same scores (copied back) must give the same indices
    w = wl.Workload("p", "bf16", H=4, d=128, W=1, n_c=50, B=1500, L_k=2345, seed=33, sigma=0.5, keys="clustered")
    Q_obs, K, V = wl.candidates(w)
    got = ctx.kv_score(dev(Q_obs), dev(K))
    sel = ctx.kv_select_compact(got["score"], w.B, dev(K), dev(V))
    torch.cuda.synchronize()
    want = oracle.kv_select_compact(got["score"].cpu().numpy(), w.B, wl.bits(K), wl.bits(V))
    assert np.array_equal(sel["kept_idx"].cpu().numpy(), want["kept_idx"])
    assert np.array_equal(wl.bits(sel["K_dst"].cpu()), want["K_dst"])
    # information only: overlap with the fully-oracle pipeline
    full = oracle.kv_select_compact(oracle.kv_score(wl.bits(Q_obs), wl.bits(K))["score"], w.B)
    overlap = np.mean([len(set(a) & set(b)) / w.B for a, b in zip(full["kept_idx"], want["kept_idx"])])
    assert overlap > 0.99


# ------------------------------------------------------------------------------------ canaries

class _Guarded:
    """Device buffers with canary elements in front of and behind the part a call may write."""

    def __init__(self):
        self.bufs = []

    def flat(self, n, dtype, pad=64, fill=0):
        buf = torch.full((n + 2 * pad,), 113, dtype=dtype, device="cuda")
        buf[pad:pad + n] = fill
        self.bufs.append((buf, pad, n))
        return buf[pad:pad + n]

    def rows(self, H, R, d, dtype):
        """[H, R, d] view with one canary row before and after every head's rows."""
        buf = torch.full((H, R + 2, d), 113, dtype=dtype, device="cuda")
        self.bufs.append((buf, None, R))
        return buf[:, 1:R + 1]

    def check(self):
        for buf, pad, n in self.bufs:
            if pad is None:
                assert (buf[:, 0] == 113).all() and (buf[:, n + 1] == 113).all()
            else:
                assert (buf[:pad] == 113).all() and (buf[pad + n:] == 113).all()


def test_outputs_stay_inside_their_buffers(ctx):
    # every output of every call sits between canaries, on ragged sizes (nothing a multiple of a tile)
    g = _Guarded()
    w = wl.Workload("c", "bf16", H=3, d=128, W=3, n_c=333, B=211, L_k=544, seed=77, sigma=0.5, keys="clustered")
    n_el = w.n_c * w.hidden
    off = np.arange(w.W + 1, dtype=np.int64) * n_el
    cur, prev = wl.indicator_pair(w.W, n_el, [0.3, 0.01, 0.3], 5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dec = ctx.chunk_decide(dev(cur), dev(prev), off, i32([4] * w.W), 1, 0.1, g.flat(w.W, torch.float32),
                           l1rel=g.flat(w.W, torch.float32), recompute=g.flat(w.W, torch.uint8),
                           active_ids=g.flat(w.W, torch.int32), n_active=g.flat(1, torch.int32), status=status)
    y, cache = g.flat(w.W * n_el, torch.bfloat16), g.flat(w.W * n_el, torch.bfloat16)
    ctx.chunk_cache_apply(dev(cur), y, cache, off, dec["recompute"], status=status)
    Q, K, V = wl.qkv(w)
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O = g.rows(w.H, w.window_rows, w.d, torch.bfloat16)
    lse = g.rows(w.H, w.window_rows, 1, torch.float32)[:, :, 0]
    ctx.chunk_attention(dev(Q), dev(K), dev(V), q_off, vis, slo, spo, dec["active_ids"], dec["n_active"], O, lse=lse,
                        status=status)
    Q_obs, Kc, Vc = wl.candidates(w)
    outs = {k: g.flat(w.H * w.L_k, torch.float32).view(w.H, w.L_k) for k in ("imp", "red", "score")}
    ctx.kv_score(dev(Q_obs), dev(Kc), status=status, **outs)
    ctx.kv_score(dev(Q_obs), dev(Kc), status=status, red_mode=1, **outs)
    kept = g.flat(w.H * w.B, torch.int32).view(w.H, w.B)
    ctx.kv_select_compact(outs["score"], w.B, dev(Kc), dev(Vc), g.rows(w.H, w.B, w.d, torch.bfloat16),
                          g.rows(w.H, w.B, w.d, torch.bfloat16), kept_idx=kept, n_kept=g.flat(1, torch.int32), status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    g.check()
    assert dec["recompute"].cpu().tolist() == [1, 0, 1] and int(kept.max().item()) < w.L_k


def test_a_wait_that_nobody_ends_gives_up_and_reports_it(ctx):
    # the bounded wait of the tensor-core kernels, made to run out on purpose: one warp waits 1 ms for a barrier that
    # is never signalled, returns, and the status word says so; the context keeps working afterwards
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx.selftest_bounded_wait(1_000_000, status, waited)
    torch.cuda.synchronize()
    assert status.item() == 1  # FC_DEV_TIMEOUT
    assert 0.9e6 <= waited.item() <= 50e6
    w = wl.CONFIGS["tiny_f32"]
    _attention_case(ctx, w, [0, 2], atol=1e-4, rel_l2=1e-4)


# ------------------------------------------------------------------------------------ error conventions

def test_bad_arguments_return_a_status_and_launch_nothing(ctx):
    import paper_2602_10825_b200 as fc
    w = wl.CONFIGS["tiny_f32"]
    Q, K, V = (dev(t) for t in wl.qkv(w))
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O = torch.zeros_like(Q)
    act, n_act = i32([0, 1, 2, 3]), i32([4])
    with pytest.raises(fc.FcError, match="workspace"):
        ctx.chunk_decide(Q.view(-1), K.view(-1)[:Q.numel()], [0, Q.numel()], i32([0]), 1, 0.1,
                         torch.zeros(1, device="cuda"), ws=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(fc.FcError, match="unsupported"):
        ctx.chunk_attention(Q[:, :, :48].contiguous(), K[:, :, :48].contiguous(), V[:, :, :48].contiguous(),
                            q_off, vis, slo, spo, act, n_act, O[:, :, :48].contiguous())
    with pytest.raises(fc.FcError, match="aligned"):
        Qm = torch.zeros(Q.numel() + 4, device="cuda")[1:1 + Q.numel()].view_as(Q)  # base off by 4 bytes
        ctx.chunk_attention(Qm, K, V, q_off, vis, slo, spo, act, n_act, O)
    with pytest.raises(fc.FcError, match="invalid"):
        ctx.kv_score(Q[:, :50], K, pool_k=4)
    with pytest.raises(fc.FcError, match="invalid"):  # the cache must be a tensor of its own
        flat = Q.view(-1)
        ctx.chunk_cache_apply(flat, flat.clone(), flat, [0, flat.numel()], torch.zeros(1, dtype=torch.uint8, device="cuda"))
    with pytest.raises(fc.FcError, match="invalid"):
        ctx.chunk_decide(Q.view(-1), K.view(-1)[:Q.numel()], [0, Q.numel()], i32([0]), 1, 0.1,
                         torch.zeros(1, device="cuda"), policy=7)
    with pytest.raises(fc.FcError, match="invalid"):
        bad_vis = vis.copy()
        bad_vis[-1] += 1  # beyond the logical length
        ctx.chunk_attention(Q, K, V, q_off, bad_vis, slo, spo, act, n_act, O)
    torch.cuda.synchronize()
    assert (O == 0).all()
