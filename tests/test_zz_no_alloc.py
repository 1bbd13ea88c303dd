"""The no-allocation entry point fc_chunk_decide_static against fc_chunk_decide and against the CPU oracle.

Some callers cannot allocate device memory where they call the library (inside an allocator or
memory-pool callback, in a loop that must stay off the allocator, or when another runtime owns all
device memory and hands out fixed buffers), so they have no workspace to give.  For them the
decision kernel has a twin whose scratch is a fixed 1 MiB array inside the library.  This test
calls the twin through the C ABI twice in a row (the array keeps the first call's contents) and
checks both results against the workspace-taking entry point on the same inputs, and first-hand
against the oracle's statement of Eqs. 5 and 8.  It is collected last so that a run stopping at the
first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


def _outputs(n):
    return dict(l1rel=torch.full((n,), -1.0, device="cuda"), recompute=torch.full((n,), 9, dtype=torch.uint8, device="cuda"),
                active_ids=torch.full((n,), -7, dtype=torch.int32, device="cuda"),
                n_active=torch.full((1,), -7, dtype=torch.int32, device="cuda"))


def test_static_scratch_decide_matches_workspace_decide_twice():
    import paper_2602_10825_b200 as fc
    from paper_2602_10825_b200 import build as fc_build
    fc_build.build()
    ctx = fc.Context(0)
    assert fc.lib().fc_chunk_decide_static_max_bytes() == 1 << 20
    # two different problems back to back: the second must not be disturbed by what the first left
    cases = [([40000, 8192 * 5 + 24, 123456], [0.05, 0.2, 0.4], torch.bfloat16, 0.15, 11),
             ([4096 * 7, 999], [0.3, 0.01], torch.float32, 0.1, 12)]
    for lens, target, dtype, eps, seed in cases:
        parts = [wl.indicator_pair(1, L, [r], seed * 10 + i, dtype=dtype) for i, (L, r) in enumerate(zip(lens, target))]
        cur_h, prev_h = torch.cat([p[0] for p in parts]), torch.cat([p[1] for p in parts])
        cur, prev = cur_h.cuda(), prev_h.cuda()
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        n = len(lens)
        step = torch.full((n,), 3, dtype=torch.int32, device="cuda")
        acc0 = torch.linspace(0.0, 0.05, n, device="cuda")
        acc_ref, acc_new = acc0.clone(), acc0.clone()
        ref = ctx.chunk_decide(cur, prev, off, step, 1, eps, acc_ref, **_outputs(n))
        new = ctx.chunk_decide_static(cur, prev, off, step, 1, eps, acc_new, **_outputs(n))
        torch.cuda.synchronize()
        # same kernels, same fixed summation order: the integer outputs match exactly and the
        # floating-point ones to the tolerance the decide parity tests use (they are in fact equal)
        assert torch.equal(new["recompute"], ref["recompute"])
        assert torch.equal(new["active_ids"], ref["active_ids"])
        assert torch.equal(new["n_active"], ref["n_active"])
        np.testing.assert_allclose(new["l1rel"].cpu().numpy(), ref["l1rel"].cpu().numpy(), rtol=2e-6)
        np.testing.assert_allclose(acc_new.cpu().numpy(), acc_ref.cpu().numpy(), rtol=4e-6, atol=1e-9)
        assert int(ref["n_active"].item()) >= 1
        # and against the oracle itself: decisions bit-exact, no chunk within the guard band of the threshold
        want = oracle.chunk_decide(wl.bits(cur_h), wl.bits(prev_h), off, np.full(n, 3, np.int32), 1, eps,
                                   acc0.cpu().numpy())
        assert np.abs(acc0.cpu().numpy() + want["l1rel"] - eps).min() > 1e-3 * eps
        assert new["recompute"].cpu().numpy().tolist() == want["recompute"].tolist()
        assert int(new["n_active"].item()) == want["n_active"]
        assert new["active_ids"].cpu().numpy()[:want["n_active"]].tolist() == want["active_ids"].tolist()
        np.testing.assert_allclose(new["l1rel"].cpu().numpy(), want["l1rel"], rtol=2e-6)
        np.testing.assert_allclose(acc_new.cpu().numpy(), want["acc"], rtol=4e-6, atol=1e-9)
    # a problem whose slab pairs would not fit the array is refused, and nothing is launched
    big = 300_000_000
    out = _outputs(1)
    with pytest.raises(fc.FcError, match="built-in scratch"):
        ctx.chunk_decide_static(cur, prev, [0, big], torch.zeros(1, dtype=torch.int32, device="cuda"), 1, 0.1,
                                torch.zeros(1, device="cuda"), **out)
    torch.cuda.synchronize()
    assert int(out["n_active"].item()) == -7
    ctx.close()
