"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test compares the oracle with something it does not itself compute: hand-worked fixtures,
closed forms, invariants, or library routines (torch CPU fp64) for the special cases that reduce
to them.  A dropped term, a wrong sign or index, or a transposed operand fails at least one.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads as wl


# --------------------------------------------------------------------------- decide (Eqs. 5, 8)

def _decide_sequence(r_seq, eps, m, n_elem=4096, seed=11):
    """Run one chunk through the rule with constructed inputs whose indicator is r_seq[s]."""
    acc = np.zeros(1, np.float32)
    flags, accs, rs = [], [], []
    for s, r in enumerate(r_seq):
        cur, prev = wl.indicator_pair(1, n_elem, [r], seed + s, dtype=torch.float32)
        out = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), [0, n_elem], [s], m, eps, acc)
        acc = out["acc"]
        flags.append(int(out["recompute"][0]))
        accs.append(float(acc[0]))
        rs.append(float(out["l1rel"][0]))
    return flags, accs, rs


def test_decide_hand_trace(golden):
    g = golden("decide_hand_trace.txt")
    flags, accs, rs = _decide_sequence(g["r"], g["eps"][0], int(g["warmup_m"][0]))
    assert flags == [int(x) for x in g["recompute"]]
    np.testing.assert_allclose(accs, g["acc_after"], atol=2e-6)
    np.testing.assert_allclose(rs, g["r"], rtol=1e-5)


def test_decide_indicator_closed_form_and_denominator_is_previous_state():
    # prev = 1 everywhere, cur = 1.5 everywhere: sum|cur-prev| / sum|prev| = 0.5 (not 1/3, which a
    # denominator taken from the later state would give).
    n = 1000
    prev = np.ones(n, np.float32)
    cur = np.full(n, 1.5, np.float32)
    out = oracle.chunk_decide(cur, prev, [0, n], [5], 0, 10.0, np.zeros(1, np.float32))
    assert out["l1rel"][0] == np.float32(0.5)
    # sign of the difference must not matter (absolute values)
    cur2 = np.where(np.arange(n) % 2 == 0, 1.5, 0.5).astype(np.float32)
    out2 = oracle.chunk_decide(cur2, prev, [0, n], [5], 0, 10.0, np.zeros(1, np.float32))
    assert out2["l1rel"][0] == np.float32(0.5)


def test_decide_segments_are_independent_and_ragged():
    # three chunks of different lengths; each chunk's indicator only sees its own elements
    lens = [7, 1000, 333]
    off = np.concatenate([[0], np.cumsum(lens)])
    target = [0.25, 0.5, 0.125]
    prev = np.ones(off[-1], np.float32) * 2
    cur = prev.copy()
    for c, r in enumerate(target):
        cur[off[c]:off[c + 1]] *= (1 + r)
    out = oracle.chunk_decide(cur, prev, off, [9, 9, 9], 1, 0.3, np.array([0.1, 0.0, 0.2], np.float32))
    np.testing.assert_array_equal(out["l1rel"], np.array(target, np.float32))
    # s = [.35, .5, .325] all > .3 except none -> all recompute; check with a higher eps
    out = oracle.chunk_decide(cur, prev, off, [9, 9, 9], 1, 0.4, np.array([0.1, 0.0, 0.2], np.float32))
    assert out["recompute"].tolist() == [0, 1, 0]
    assert out["active_ids"].tolist() == [1] and out["n_active"] == 1
    np.testing.assert_allclose(out["acc"], [0.35, 0.0, 0.325], rtol=1e-6)


def test_decide_threshold_is_strict_and_limits():
    n = 64
    prev = np.ones(n, np.float32)
    cur = np.full(n, 1.25, np.float32)  # r = 0.25 exactly
    z = np.zeros(1, np.float32)
    # s == eps reuses (case 3 is "<= eps"), just below eps recomputes
    assert oracle.chunk_decide(cur, prev, [0, n], [3], 1, 0.25, z)["recompute"][0] == 0
    assert oracle.chunk_decide(cur, prev, [0, n], [3], 1, np.nextafter(np.float32(0.25), np.float32(0)), z)["recompute"][0] == 1
    # eps = +inf: only warm-up steps compute; eps < 0: always compute
    assert oracle.chunk_decide(cur, prev, [0, n], [0], 1, math.inf, z)["recompute"][0] == 1
    assert oracle.chunk_decide(cur, prev, [0, n], [1], 1, math.inf, z)["recompute"][0] == 0
    assert oracle.chunk_decide(cur, prev, [0, n], [7], 1, -1.0, z)["recompute"][0] == 1
    # warm-up interval is m steps wide and resets the accumulator
    out = oracle.chunk_decide(cur, prev, [0, n], [4], 5, math.inf, np.array([0.3], np.float32))
    assert out["recompute"][0] == 1 and out["acc"][0] == 0.0
    # forced chunk (a newly initialised chunk must be computed)
    out = oracle.chunk_decide(cur, prev, [0, n], [9], 1, math.inf, z, force=[1])
    assert out["recompute"][0] == 1
    # zero denominator: +inf when something changed, 0 when nothing did; never NaN
    zero = np.zeros(n, np.float32)
    assert np.isposinf(oracle.chunk_decide(cur, zero, [0, n], [9], 1, 1.0, z)["l1rel"][0])
    assert oracle.chunk_decide(zero, zero, [0, n], [9], 1, 1.0, z)["l1rel"][0] == 0.0


def test_decide_power_of_two_scaling_is_bit_invariant():
    cur, prev = wl.indicator_pair(3, 5000, [0.03, 0.11, 0.4], 5, dtype=torch.bfloat16)
    off = [0, 5000, 10000, 15000]
    a = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), off, [2, 2, 2], 1, 0.1, np.zeros(3, np.float32))
    b = oracle.chunk_decide(wl.bits(cur * 8), wl.bits(prev * 8), off, [2, 2, 2], 1, 0.1, np.zeros(3, np.float32))
    np.testing.assert_array_equal(a["l1rel"], b["l1rel"])
    np.testing.assert_allclose(a["l1rel"], [0.03, 0.11, 0.4], rtol=2e-2)  # bf16 rounding of cur


# --------------------------------------------------------------------------- attention (Sec. 3.3)

def _tiny_attention_case(dtype=torch.float32, H=2, W=3, n_c=5, B=4, d=8, seed=3):
    w = wl.Workload("t", "f32" if dtype == torch.float32 else "bf16", H=H, d=d, W=W, n_c=n_c, B=B,
                    L_k=B + n_c, seed=seed)
    Q, K, V = wl.qkv(w)
    return w, Q, K, V, wl.prefix_layout(w)


def test_attention_matches_library_sdpa_with_block_causal_mask():
    w, Q, K, V, (q_off, vis, slo, spo) = _tiny_attention_case()
    O, lse = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1, 2])
    # library routine on the same problem: boolean mask "key j visible to row r iff j < vis[chunk(r)]"
    rows = torch.arange(w.window_rows)
    allowed = torch.arange(K.shape[1])[None, :] < torch.as_tensor(vis)[rows // w.n_c][:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(Q.double(), K.double(), V.double(), attn_mask=allowed)
    np.testing.assert_allclose(O, ref.numpy(), rtol=1e-10, atol=1e-12)
    s = (Q.double() @ K.double().transpose(1, 2)) / math.sqrt(w.d)
    s = s.masked_fill(~allowed, -math.inf)
    np.testing.assert_allclose(lse, torch.logsumexp(s, -1).numpy(), rtol=1e-12)
    # softmax rows sum to one: sum_j exp(s_j - lse) = 1
    np.testing.assert_allclose(torch.exp(s - torch.as_tensor(lse)[..., None]).sum(-1).numpy(), 1.0, rtol=1e-12)


def test_attention_brute_force_python_loops():
    w, Q, K, V, (q_off, vis, slo, spo) = _tiny_attention_case(H=1, W=2, n_c=3, B=2, d=4)
    O, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1])
    q, k, v = Q.double().numpy()[0], K.double().numpy()[0], V.double().numpy()[0]
    for r in range(w.window_rows):
        n_vis = w.B + (r // w.n_c + 1) * w.n_c
        e = [math.exp(sum(q[r][t] * k[j][t] for t in range(w.d)) / math.sqrt(w.d)) for j in range(n_vis)]
        for t in range(w.d):
            want = sum(e[j] * v[j][t] for j in range(n_vis)) / sum(e)
            assert abs(O[0, r, t] - want) < 1e-12


def test_attention_closed_forms():
    w, Q, K, V, (q_off, vis, slo, spo) = _tiny_attention_case()
    Qb, Kb, Vb = wl.bits(Q), wl.bits(K), wl.bits(V)
    # constant V rows -> output equals that constant
    Vc = np.ascontiguousarray(np.broadcast_to(np.arange(w.d, dtype=np.float32), V.shape))
    O, _ = oracle.chunk_attention(Qb, Kb, Vc, q_off, vis, slo, spo, [0, 1, 2])
    np.testing.assert_allclose(O, np.broadcast_to(np.arange(w.d), O.shape), rtol=1e-12)
    # zero queries -> uniform weights -> output is the mean of exactly the visible V rows
    O, lse = oracle.chunk_attention(np.zeros_like(Qb), Kb, Vb, q_off, vis, slo, spo, [0, 1, 2])
    for c in range(w.W):
        want = V.double().numpy()[:, :vis[c]].mean(1)
        for r in range(q_off[c], q_off[c + 1]):
            np.testing.assert_allclose(O[:, r], want, rtol=1e-12)
            np.testing.assert_allclose(lse[:, r], math.log(vis[c]), rtol=1e-12)
    # a one-token visible prefix returns that V row
    O, _ = oracle.chunk_attention(Qb, Kb, Vb, q_off, [1, 1, 1], slo, spo, [0, 1, 2])
    np.testing.assert_allclose(O, np.broadcast_to(V.double().numpy()[:, :1], O.shape), rtol=1e-12)


def test_attention_inactive_chunks_untouched_and_all_skip_identity():
    w, Q, K, V, (q_off, vis, slo, spo) = _tiny_attention_case()
    cached = np.random.default_rng(0).normal(size=(w.H, w.window_rows, w.d))
    O, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [],
                                  O_init=cached)
    assert np.array_equal(O, cached)  # all-skip: cached outputs returned unchanged, bit for bit
    O, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [1],
                                  O_init=cached)
    assert np.array_equal(O[:, :w.n_c], cached[:, :w.n_c]) and np.array_equal(O[:, 2 * w.n_c:], cached[:, 2 * w.n_c:])
    full, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1, 2])
    assert np.array_equal(O[:, w.n_c:2 * w.n_c], full[:, w.n_c:2 * w.n_c])
    # sampled rows agree with the full evaluation
    rows = [0, 4, 5, 9, 14]
    Os, lses = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1, 2],
                                      sample_rows=rows)
    assert np.array_equal(Os, full[:, rows])


def test_attention_index_maps():
    w, Q, K, V, (q_off, vis, slo, spo) = _tiny_attention_case()
    Qb = wl.bits(Q)
    base, _ = oracle.chunk_attention(Qb, wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1, 2])
    # segment table: store the clean region AFTER the window physically; logical order unchanged
    L = K.shape[1]
    perm_phys = np.concatenate([np.arange(w.B, L), np.arange(0, w.B)])  # new physical order of old rows
    K2, V2 = K[:, perm_phys].contiguous(), V[:, perm_phys].contiguous()
    spo2 = np.where(spo < w.B, spo + (L - w.B), spo - w.B).astype(np.int32)
    O2, _ = oracle.chunk_attention(Qb, wl.bits(K2), wl.bits(V2), q_off, vis, slo, spo2, [0, 1, 2])
    assert np.array_equal(O2, base)
    # token-level map on a shuffled physical store == attention on the ordered store
    rng = np.random.default_rng(1)
    tok = np.stack([rng.permutation(L) for _ in range(w.H)]).astype(np.int32)  # logical j -> physical row
    K3, V3 = torch.empty_like(K), torch.empty_like(V)
    for h in range(w.H):
        K3[h, tok[h]] = K[h]
        V3[h, tok[h]] = V[h]
    O3, _ = oracle.chunk_attention(Qb, wl.bits(K3), wl.bits(V3), q_off, vis, None, None, [0, 1, 2],
                                   kv_token_index=tok)
    assert np.array_equal(O3, base)
    # permuting the visible rows of K and V together (inside the clean region) changes nothing
    p = np.arange(L)
    p[:w.B] = p[:w.B][::-1]
    O4, _ = oracle.chunk_attention(Qb, wl.bits(K[:, p].contiguous()), wl.bits(V[:, p].contiguous()),
                                   q_off, vis, slo, spo, [0, 1, 2])
    np.testing.assert_allclose(O4, base, rtol=1e-12, atol=1e-14)


def test_attention_gqa_and_bf16_inputs():
    w = wl.Workload("g", "bf16", H=4, d=8, W=2, n_c=4, B=3, L_k=7, seed=9)
    Q, K, V = wl.qkv(w)
    K, V = K[:2].contiguous(), V[:2].contiguous()  # 2 kv heads, group of 2 query heads each
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(K), wl.bits(V), q_off, vis, slo, spo, [0, 1], H_kv=2)
    rows = torch.arange(w.window_rows)
    allowed = torch.arange(K.shape[1])[None, :] < torch.as_tensor(vis)[rows // w.n_c][:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(
        Q.double(), K.double().repeat_interleave(2, 0), V.double().repeat_interleave(2, 0), attn_mask=allowed)
    np.testing.assert_allclose(O, ref.numpy(), rtol=1e-10, atol=1e-12)


# --------------------------------------------------------------------------- scores (Eqs. 9-12)

def _torch_scores(Q, K, lam, pool_k, group=1):
    """The same quantities from library routines (torch CPU, fp64)."""
    Qd, Kd = Q.double(), K.double()
    d = Q.shape[-1]
    Kq = Kd.repeat_interleave(group, 0)
    p = torch.softmax(Qd @ Kq.transpose(1, 2) / math.sqrt(d), dim=-1)  # softmax over keys
    imp = p.mean(1).reshape(K.shape[0], group, -1).mean(1)
    pooled = torch.nn.functional.max_pool1d(imp[:, None], kernel_size=pool_k, stride=1, padding=pool_k // 2)[:, 0]
    kh = torch.nn.functional.normalize(Kd, dim=-1, eps=1e-12)
    S = kh @ kh.transpose(1, 2)
    S = S - torch.diag_embed(torch.diagonal(S, dim1=1, dim2=2))
    red = torch.softmax(S.mean(1), dim=-1)
    return imp, pooled, red, lam * pooled - (1 - lam) * red


def test_score_worked_example(golden):
    g = golden("score_worked_example.txt")
    K = np.asarray(g["keys"], np.float32).reshape(1, 6, 2)
    Q = np.asarray(g["queries"], np.float32).reshape(1, 2, 2)
    for mode in (oracle.RED_PLAIN, oracle.RED_MEANKEY):
        out = oracle.kv_score(Q, K, lambda_=0.07, pool_k=3, red_mode=mode)
        np.testing.assert_allclose(out["imp"][0], g["imp"], atol=1e-6)
        np.testing.assert_allclose(out["imp_pooled"][0], g["pooled"], atol=1e-6)
        np.testing.assert_allclose(out["red"][0], g["red"], atol=1e-6)
        np.testing.assert_allclose(out["score"][0], g["score"], atol=1e-6)
        assert out["score"][0][0] == out["score"][0][1]  # duplicated key: exact tie
    sc = oracle.kv_score(Q, K, lambda_=0.07, pool_k=3)["score"]
    for B, key in ((3, "kept_B3"), (2, "kept_B2"), (6, "kept_B6"), (9, "kept_B6")):
        kept = oracle.kv_select_compact(sc, B)["kept_idx"][0]
        assert kept.tolist() == [int(x) for x in g[key]]


@pytest.mark.parametrize("dtype,group", [(torch.float32, 1), (torch.bfloat16, 1), (torch.float32, 2)])
def test_score_matches_library_routines(dtype, group):
    H_kv, L_q, L_k, d = 2, 5, 37, 16
    Q = wl.normal((H_kv * group, L_q, d), 21, 1.0, dtype)
    K = wl.normal((H_kv, L_k, d), 22, 1.0, dtype)
    imp, pooled, red, score = _torch_scores(Q, K, 0.3, 5, group)
    for mode in (oracle.RED_PLAIN, oracle.RED_MEANKEY):
        out = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=0.3, pool_k=5, red_mode=mode)
        np.testing.assert_allclose(out["imp"], imp.numpy(), rtol=1e-10)
        np.testing.assert_allclose(out["imp_pooled"], pooled.numpy(), rtol=1e-10)
        np.testing.assert_allclose(out["red"], red.numpy(), rtol=1e-10)
        np.testing.assert_allclose(out["score"], score.float().numpy(), rtol=2e-6, atol=1e-9)
        np.testing.assert_allclose(out["imp"].sum(1), 1.0, rtol=1e-12)  # distributions over tokens
        np.testing.assert_allclose(out["red"].sum(1), 1.0, rtol=1e-12)


def test_score_plain_definition_equals_meankey_identity():
    Q = wl.normal((3, 4, 32), 31)
    K = wl.normal((3, 200, 32), 32)
    K[1, 17] = 0  # a zero key: normalisation guard, and the identity must still hold
    a = oracle.kv_score(wl.bits(Q), wl.bits(K), red_mode=oracle.RED_PLAIN)
    b = oracle.kv_score(wl.bits(Q), wl.bits(K), red_mode=oracle.RED_MEANKEY)
    np.testing.assert_allclose(a["red"], b["red"], rtol=1e-12, atol=1e-15)
    assert np.array_equal(a["score"], b["score"])


def test_score_closed_forms():
    K = wl.normal((1, 30, 8), 41)
    # zero queries: every key gets the same attention weight, Imp = 1 / L_k
    out = oracle.kv_score(np.zeros((1, 3, 8), np.float32), wl.bits(K))
    np.testing.assert_allclose(out["imp"], 1 / 30, rtol=1e-12)
    # identical keys: identical redundancy, Red = 1 / L_k
    K_same = np.ascontiguousarray(np.broadcast_to(wl.bits(K)[:, :1], (1, 30, 8)))
    out = oracle.kv_score(np.ones((1, 3, 8), np.float32), K_same)
    np.testing.assert_allclose(out["red"], 1 / 30, rtol=1e-12)
    # lambda = 1 -> score is the pooled importance; lambda = 0 -> minus the redundancy
    Q = wl.normal((1, 3, 8), 42)
    o1 = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=1.0, pool_k=1)
    np.testing.assert_allclose(o1["score"], o1["imp"].astype(np.float32), rtol=1e-6)
    o0 = oracle.kv_score(wl.bits(Q), wl.bits(K), lambda_=0.0)
    np.testing.assert_allclose(o0["score"], -o0["red"].astype(np.float32), rtol=1e-6)
    # one dominant key: importance concentrates there and pooling spreads it over the window
    Kd = np.zeros((1, 30, 8), np.float32)
    Kd[0, 12, 0] = 100.0
    Qd = np.zeros((1, 2, 8), np.float32)
    Qd[0, :, 0] = 10.0
    o = oracle.kv_score(Qd, Kd, pool_k=5)
    assert abs(o["imp"][0, 12] - 1.0) < 1e-9
    np.testing.assert_allclose(o["imp_pooled"][0, 10:15], 1.0, rtol=1e-9)
    assert o["imp_pooled"][0, 9] < 1e-9 and o["imp_pooled"][0, 15] < 1e-9


def test_score_accumulation_over_steps_is_the_mean():
    K = wl.normal((2, 40, 16), 51)
    Qs = [wl.normal((2, 6, 16), 52 + s) for s in range(3)]
    singles = [oracle.kv_score(wl.bits(q), wl.bits(K))["imp"] for q in Qs]
    acc = np.zeros((2, 40), np.float64)
    oracle.kv_score(wl.bits(Qs[0]), wl.bits(K), imp_accum=acc, accum_phase=1, n_steps=3)
    oracle.kv_score(wl.bits(Qs[1]), wl.bits(K), imp_accum=acc, accum_phase=1, n_steps=3)
    out = oracle.kv_score(wl.bits(Qs[2]), wl.bits(K), imp_accum=acc, accum_phase=2, n_steps=3)
    np.testing.assert_allclose(out["imp"], sum(singles) / 3, rtol=1e-12)
    np.testing.assert_allclose(out["imp"].sum(1), 1.0, rtol=1e-12)


# --------------------------------------------------------------------------- select + compact

def test_select_matches_full_sort_and_topk():
    rng = np.random.default_rng(7)
    score = rng.normal(size=(3, 500)).astype(np.float32)
    score[:, ::7] = score[:, 3:4]  # many exact ties
    score[1, 5] = np.nan
    score[2, 11] = -0.0
    score[2, 12] = 0.0
    for B in (1, 2, 37, 499, 500, 700):
        out = oracle.kv_select_compact(score, B)
        n_keep = min(B, 500)
        assert out["n_kept"] == n_keep
        for h in range(3):
            s = np.where(np.isnan(score[h]), -np.inf, score[h])
            order = sorted(range(500), key=lambda j: (-s[j], j))  # textbook full sort
            assert out["kept_idx"][h].tolist() == sorted(order[:n_keep])
    # B = 1 is the arg-max with the lowest index among equals
    tie = np.array([[1.0, 3.0, 3.0, 2.0]], np.float32)
    assert oracle.kv_select_compact(tie, 1)["kept_idx"].tolist() == [[1]]
    # distinct scores: same set as the library top-k
    distinct = rng.permutation(1000).astype(np.float32).reshape(2, 500)
    kept = oracle.kv_select_compact(distinct, 123)["kept_idx"]
    ref = torch.topk(torch.from_numpy(distinct), 123, dim=1).indices.sort(1).values.numpy()
    assert np.array_equal(kept, ref)


def test_compact_copies_rows_and_budget_identity():
    w = wl.Workload("c", "bf16", H=3, d=16, W=1, n_c=8, B=20, L_k=50, seed=5)
    _, K, V = wl.candidates(w)
    score = np.random.default_rng(3).normal(size=(3, 50)).astype(np.float32)
    out = oracle.kv_select_compact(score, 20, wl.bits(K), wl.bits(V))
    for h in range(3):
        assert np.array_equal(out["K_dst"][h], wl.bits(K)[h][out["kept_idx"][h]])
        assert np.array_equal(out["V_dst"][h], wl.bits(V)[h][out["kept_idx"][h]])
        assert np.all(np.diff(out["kept_idx"][h]) > 0)
    # budget >= cache length: compression is the identity
    ident = oracle.kv_select_compact(score, 50, wl.bits(K), wl.bits(V))
    assert np.array_equal(ident["kept_idx"], np.broadcast_to(np.arange(50), (3, 50)))
    assert np.array_equal(ident["K_dst"], wl.bits(K)) and np.array_equal(ident["V_dst"], wl.bits(V))
    # permuting the candidate rows permutes the kept set accordingly (distinct scores)
    perm = np.random.default_rng(4).permutation(50)
    out_p = oracle.kv_select_compact(score[:, perm], 20)
    for h in range(3):
        assert sorted(perm[out_p["kept_idx"][h]].tolist()) == out["kept_idx"][h].tolist()


def test_attention_on_compacted_cache_equals_token_map_on_uncompacted():
    # Compressing the clean region and attending to the compact copy must equal attending to the
    # original store through the kept-index map.
    w = wl.Workload("m", "f32", H=2, d=8, W=2, n_c=4, B=6, L_k=10, seed=8)
    Q, K, V = wl.qkv(w)  # physical [10 candidates + ... ] we treat the first L_k rows as candidates
    L_phys = K.shape[1]
    score = np.random.default_rng(5).normal(size=(2, w.B + 0 + 4)).astype(np.float32)  # 10 candidates
    sel = oracle.kv_select_compact(score, w.B, wl.bits(K[:, :10].contiguous()), wl.bits(V[:, :10].contiguous()))
    # compact store: [kept 6 | window 8 rows taken from physical rows 6..13 of the original]
    Kc = torch.cat([torch.from_numpy(sel["K_dst"]), K[:, 6:]], 1).contiguous()
    Vc = torch.cat([torch.from_numpy(sel["V_dst"]), V[:, 6:]], 1).contiguous()
    q_off, vis, slo, spo = wl.prefix_layout(w)
    O_compact, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(Kc), wl.bits(Vc), q_off, vis, slo, spo, [0, 1])
    # uncompacted store: candidates (10 rows) followed by the same window rows
    Ku = torch.cat([K[:, :10], K[:, 6:]], 1).contiguous()
    Vu = torch.cat([V[:, :10], V[:, 6:]], 1).contiguous()
    tok = np.concatenate([sel["kept_idx"], np.broadcast_to(np.arange(10, 10 + 8, dtype=np.int32), (2, 8))], 1)
    O_map, _ = oracle.chunk_attention(wl.bits(Q), wl.bits(Ku), wl.bits(Vu), q_off, vis, None, None, [0, 1],
                                      kv_token_index=tok)
    assert np.array_equal(O_compact, O_map)
    assert L_phys == 14


# --------------------------------------------------------------------------- uniform policy (caption of Fig. 3)

def test_uniform_policy_hand_trace(golden):
    g = golden("uniform_policy_hand_trace.txt")
    eps, m, n_el = g["eps"][0], int(g["warmup_m"][0]), 4096
    acc = np.zeros(3, np.float32)
    for s in range(len(g["acc_after"])):
        target = [g["r_chunk0"][s], g["r_chunk1"][s], g["r_chunk2"][s]]
        # |prev| = 1 everywhere (random signs), cur = prev (1 +- r): equal weights, so the indicator over several
        # chunks taken as one tensor is the mean of the chunks' own indicators
        prev = torch.sign(wl.normal((3 * n_el,), 40 + s)) + 0.0
        prev[prev == 0] = 1.0
        alt = torch.where(torch.arange(3 * n_el) % 2 == 0, 1.0, -1.0)
        cur = prev * (1 + torch.tensor(target, dtype=torch.float32).repeat_interleave(n_el) * alt)
        step = np.array([s, s, int(g["step_chunk2"][s])], np.int32)
        out = oracle.chunk_decide_uniform(wl.bits(cur.float()), wl.bits(prev.float()), [0, n_el, 2 * n_el, 3 * n_el],
                                          step, m, eps, acc)
        want = [int(g[f"recompute{c}"][s]) for c in range(3)]
        assert out["recompute"].tolist() == want, f"step {s}"
        assert out["active_ids"].tolist() == [c for c in range(3) if want[c]]
        np.testing.assert_allclose(out["acc"], [g["acc_after"][s]] * 3, atol=2e-6)
        acc = out["acc"]


def test_uniform_policy_reduces_to_the_chunkwise_rule_for_one_chunk_and_differs_for_several():
    # one chunk: the shared decision IS the chunk's decision (Eq. 8)
    acc_u = acc_c = np.zeros(1, np.float32)
    for s, r in enumerate([0.08, 0.05, 0.04, 0.09, 0.20, 0.01, 0.13, 0.02]):
        cur, prev = wl.indicator_pair(1, 2048, [r], 70 + s, dtype=torch.float32)
        u = oracle.chunk_decide_uniform(wl.bits(cur), wl.bits(prev), [0, 2048], [s], 1, 0.15, acc_u)
        c = oracle.chunk_decide(wl.bits(cur), wl.bits(prev), [0, 2048], [s], 1, 0.15, acc_c)
        assert u["recompute"].tolist() == c["recompute"].tolist()
        np.testing.assert_array_equal(u["acc"], c["acc"])
        np.testing.assert_array_equal(u["l1rel"], c["l1rel"])
        acc_u, acc_c = u["acc"], c["acc"]
    # several chunks: one flag for all sharing chunks, whatever their own indicators; a forced chunk computes anyway
    # and its elements do not enter the shared indicator
    n = 1000
    prev = np.ones(3 * n, np.float32)
    cur = prev.copy()
    cur[:n] *= 1.5       # chunk 0 changed by 0.5
    cur[2 * n:] *= 3.0   # chunk 2 changed by 2.0 but is forced: excluded from the shared sum
    out = oracle.chunk_decide_uniform(cur, prev, [0, n, 2 * n, 3 * n], [5, 5, 5], 1, 0.3, np.zeros(3, np.float32),
                                      force=[0, 0, 1])
    assert out["l1rel"].tolist() == [0.25, 0.25, 2.0]   # (0.5 n + 0) / 2n for the sharing chunks
    assert out["recompute"].tolist() == [0, 0, 1]        # 0.25 <= 0.3: the sharing chunks reuse
    np.testing.assert_array_equal(out["acc"], np.float32([0.25, 0.25, 0.25]))
    out = oracle.chunk_decide_uniform(cur, prev, [0, n, 2 * n, 3 * n], [5, 5, 5], 1, 0.2, np.zeros(3, np.float32),
                                      force=[0, 0, 1])
    assert out["recompute"].tolist() == [1, 1, 1] and out["acc"].tolist() == [0.0, 0.0, 0.0]
    # the shared indicator is the ratio of the sums, not the mean of the ratios: chunks of different magnitude
    prev2 = np.concatenate([np.ones(n, np.float32), np.full(n, 9.0, np.float32)])
    cur2 = np.concatenate([np.full(n, 2.0, np.float32), np.full(n, 9.0, np.float32)])  # r0 = 1, r1 = 0
    out = oracle.chunk_decide_uniform(cur2, prev2, [0, n, 2 * n], [5, 5], 1, 10.0, np.zeros(2, np.float32))
    assert out["l1rel"].tolist() == [np.float32(0.1)] * 2  # n / (n + 9 n), not (1 + 0) / 2
    # every chunk forced or warming up: all compute, accumulator cleared
    out = oracle.chunk_decide_uniform(cur2, prev2, [0, n, 2 * n], [0, 9], 1, 10.0, np.float32([0.3, 0.3]), force=[0, 1])
    assert out["recompute"].tolist() == [1, 1] and out["acc"].tolist() == [0.0, 0.0]


# --------------------------------------------------------------------------- activation cache (Sec. 3.2)

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_cache_apply_hand_example(golden, dtype):
    g = golden("cache_apply_hand_example.txt")
    t = lambda k: wl.bits(torch.tensor(g[k], dtype=torch.float32).to(dtype))
    back = lambda a: (torch.from_numpy(a.copy()).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)).float().tolist()
    off = [0, 3, 6]
    y, cache = oracle.chunk_cache_apply(t("xA"), t("yA"), wl.bits(torch.full((6,), 77.0).to(dtype)), off, [1, 1])
    assert back(cache) == g["cacheA"] and back(y) == g["yA"]        # computed chunks: y untouched, cache = y - x
    y, cache = oracle.chunk_cache_apply(t("xB"), t("yB_in"), cache, off, [int(v) for v in g["recB"]])
    assert back(y) == g["yB_out"] and back(cache) == g["cacheB"]


def test_cache_apply_matches_library_arithmetic_and_rounding():
    # fp32 add / subtract by numpy, rounding to bf16 by torch (round to nearest even): library routines
    n = 5000
    x, yv, c = (wl.normal((2 * n,), 300 + i, 3.0, torch.bfloat16) for i in range(3))
    y, cache = oracle.chunk_cache_apply(wl.bits(x), wl.bits(yv), wl.bits(c), [0, n, 2 * n], [0, 1])
    want_y = (x.float()[:n] + c.float()[:n]).to(torch.bfloat16)
    want_c = (yv.float()[n:] - x.float()[n:]).to(torch.bfloat16)
    assert np.array_equal(y[:n], wl.bits(want_y)) and np.array_equal(y[n:], wl.bits(yv)[n:])
    assert np.array_equal(cache[n:], wl.bits(want_c)) and np.array_equal(cache[:n], wl.bits(c)[:n])
    # ties round to even: 1 + 2^-8 is halfway between two bf16 values around 1 -> 1.0; 1 + 3 * 2^-8 -> 1 + 2^-6
    xs = torch.tensor([1.0, 1.0], dtype=torch.bfloat16)
    cs = torch.tensor([2.0 ** -8, 3 * 2.0 ** -8], dtype=torch.bfloat16)
    y, _ = oracle.chunk_cache_apply(wl.bits(xs), wl.bits(xs), wl.bits(cs), [0, 2], [0])
    assert torch.from_numpy(y.copy()).view(torch.bfloat16).float().tolist() == [1.0, 1.0 + 2.0 ** -6]
    # fp32 storage: plain fp32 arithmetic, bit for bit
    xf, yf, cf = (wl.normal((n,), 310 + i, 2.0) for i in range(3))
    y, cache = oracle.chunk_cache_apply(xf.numpy(), yf.numpy(), cf.numpy(), [0, n // 2, n], [1, 0])
    assert np.array_equal(cache[:n // 2], (yf - xf).numpy()[:n // 2])
    assert np.array_equal(y[n // 2:], (xf + cf).numpy()[n // 2:])
    # a zero residual serves the input back unchanged; an empty chunk is fine
    y, _ = oracle.chunk_cache_apply(xf.numpy(), yf.numpy(), np.zeros(n, np.float32), [0, 0, n], [0, 0])
    assert np.array_equal(y, xf.numpy())


# --------------------------------------------------------------------------- similarity statistics beyond Eq. 11

def test_max_similarity_mode_against_library_routines_and_closed_forms():
    # torch fp64: normalise, cosine matrix, diagonal excluded, column maximum, softmax over tokens
    H, L, d = 2, 60, 16
    K = wl.normal((H, L, d), 801, 1.0)
    K[1, 7] = K[1, 3] * 2.5          # a duplicated direction: both tokens get similarity 1
    Q = wl.normal((H, 5, d), 802, 1.0)
    out = oracle.kv_score(Q.numpy(), K.numpy(), red_mode=oracle.RED_MAXSIM, lambda_=0.0)
    Kh = torch.nn.functional.normalize(K.double(), dim=-1)
    S = Kh @ Kh.transpose(1, 2)
    S[:, torch.arange(L), torch.arange(L)] = -float("inf")
    a = S.max(dim=1).values
    np.testing.assert_allclose(out["red"], torch.softmax(a, dim=-1).numpy(), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(oracle.key_similarity_columns(K.numpy(), np.arange(L), oracle.RED_MAXSIM), a.numpy(),
                               rtol=1e-12, atol=1e-15)
    assert abs(a[1, 7].item() - 1.0) < 1e-12 and abs(a[1, 3].item() - 1.0) < 1e-12
    # mutually orthogonal keys: every maximum is 0 -> uniform Red; the mean-based Eq. 11 gives uniform Red too
    E = torch.eye(8).reshape(1, 8, 8) * torch.arange(1, 9).reshape(1, 8, 1)
    out = oracle.kv_score(Q[:1, :, :8].contiguous().numpy(), E.numpy(), red_mode=oracle.RED_MAXSIM)
    np.testing.assert_allclose(out["red"], np.full((1, 8), 1 / 8), rtol=1e-12)
    # the maximum is never below the mean of the other columns' similarities, and differs from it in general
    mean_cols = oracle.key_similarity_columns(K.numpy(), np.arange(L), oracle.RED_PLAIN)
    assert (a.numpy() >= mean_cols * L / (L - 1) - 1e-12).all() and np.abs(a.numpy() - mean_cols).max() > 0.1


def test_similarity_columns_match_the_full_matrix_and_the_mean_key_identity():
    # sampled columns of the plain definition = the same columns of the full evaluation (both red modes of
    # kv_score), also for bf16 storage, a zero key and strided sampling
    H, L, d = 3, 130, 32
    K = wl.normal((H, L, d), 811, 0.7, torch.bfloat16)
    K[2, 11] = 0
    Q = wl.normal((H, 4, d), 812, 0.7, torch.bfloat16)
    cols = np.array([0, 1, 11, 64, 129], np.int32)
    a_cols = oracle.key_similarity_columns(wl.bits(K), cols, oracle.RED_PLAIN)
    Kh = K.double() / K.double().norm(dim=-1, keepdim=True).clamp_min(1e-12)
    S = Kh @ Kh.transpose(1, 2)
    S[:, torch.arange(L), torch.arange(L)] = 0.0
    np.testing.assert_allclose(a_cols, S.mean(dim=1)[:, cols].numpy(), rtol=1e-12, atol=1e-15)
    # and Red of the two modes of kv_score is the softmax of exactly these arguments
    full = oracle.key_similarity_columns(wl.bits(K), np.arange(L), oracle.RED_PLAIN)
    for mode in (oracle.RED_PLAIN, oracle.RED_MEANKEY):
        red = oracle.kv_score(wl.bits(Q), wl.bits(K), red_mode=mode)["red"]
        np.testing.assert_allclose(red, torch.softmax(torch.from_numpy(full), dim=-1).numpy(), rtol=1e-10)


# --------------------------------------------------------------------------- selection by units, protected tail

def test_select_units_hand_example(golden):
    g = golden("select_units_hand_example.txt")
    score = np.array([g["score"]], np.float32)
    for n_protect, key in ((0, "kept_p0"), (2, "kept_p2"), (4, "kept_p4")):
        out = oracle.kv_select_units(score, 6, unit=3, n_protect=n_protect)
        assert out["kept_idx"][0].tolist() == [int(v) for v in g[key]] and out["n_kept"] == 6


def test_select_units_reduce_to_the_token_level_selection_and_match_a_library_topk():
    rng = np.random.default_rng(17)
    score = rng.normal(size=(3, 240)).astype(np.float32)
    score[0, ::7] = score[0, 3]   # ties
    score[1, 11] = np.nan
    # unit 1, nothing protected: exactly the token-level selection
    for B in (1, 17, 239, 240, 300):
        a = oracle.kv_select_units(score, B)["kept_idx"]
        b = oracle.kv_select_compact(score, B)["kept_idx"]
        assert np.array_equal(a, b)
    # units of 8: torch's mean (fp64) and topk on distinct unit means
    s = torch.from_numpy(np.ascontiguousarray(score[2:])).double()
    means = s.reshape(1, 30, 8).mean(-1).float()
    want_units = torch.sort(torch.topk(means, 12, dim=1).indices, dim=1).values
    want = (want_units[:, :, None] * 8 + torch.arange(8)).reshape(1, -1).numpy()
    got = oracle.kv_select_units(np.ascontiguousarray(score[2:]), 96, unit=8)
    assert np.array_equal(got["kept_idx"], want) and got["n_kept"] == 96
    # a protected tail at token level: the last 5 tokens plus the best 12 of the others
    got = oracle.kv_select_units(np.ascontiguousarray(score[2:]), 17, n_protect=5)["kept_idx"][0]
    rest = np.sort(np.argsort(-score[2, :235], kind="stable")[:12])
    assert got.tolist() == rest.tolist() + [235, 236, 237, 238, 239]
    # budget at least the cache length: identity; protection beyond the budget is capped by it
    assert oracle.kv_select_units(score, 240, unit=8)["kept_idx"][0].tolist() == list(range(240))
    assert oracle.kv_select_units(score, 16, unit=8, n_protect=100)["kept_idx"][0].tolist() == list(range(224, 240))
    with pytest.raises(ValueError):
        oracle.kv_select_units(score, 100, unit=8)  # the budget must be a whole number of units
