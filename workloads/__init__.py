"""Seeded synthetic inputs shaped like FlowCache's autoregressive-video workloads.

This module only draws numbers and lays them out; it holds none of the
method's arithmetic (no indicator, no softmax, no scoring, no selection), so
both the CPU oracle's tests and the CUDA library's tests can take their inputs
from it.  Every tensor comes from a ``torch.Generator`` on the CPU with a fixed
seed and is rounded once to its storage dtype; the same bits go to both sides.

Shapes follow the paper's models: hidden width 3072 = 24 heads x 128, chunks
of 3-4 latent frames of 30 x 52 patches, cache budgets of 4-8 chunks; for the
second model family hidden width 1536 = 12 heads x 128 and blocks of 5 latent
frames of 34 x 60 patches.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
import math

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str            # "f32" | "bf16" storage type of Q/K/V and of the indicator inputs
    H: int                # attention heads (MHA: H_q = H_kv)
    d: int                # head dimension
    W: int                # chunks in the denoising window
    n_c: int              # tokens per chunk
    B: int                # clean-region budget in tokens (0 = no clean region)
    L_k: int              # candidate tokens at a compression event
    seed: int
    sigma: float = 1.0    # std of Q/K/V draws
    D: int = 0            # width of the indicator tensors per token (0 => H*d)
    eps: float = 0.15     # reuse threshold
    warmup_m: int = 1
    L_q_obs: int = 50     # observation queries (last tokens of the last window chunk)
    pool_k: int = 7
    lam: float = 0.07
    keys: str = "normal"  # "normal" | "clustered" | "ar1"
    n_steps: int = 1
    notes: str = ""

    @property
    def hidden(self) -> int:
        return self.D or self.H * self.d

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def window_rows(self) -> int:
        return self.W * self.n_c

    def attention_flops(self, active_ids) -> float:
        """4 d H n_c * sum over active chunks of the visible prefix length."""
        return 4.0 * self.d * self.H * self.n_c * sum(self.B + (i + 1) * self.n_c for i in active_ids)

    def compact_bytes(self) -> int:
        """K and V, read and write, of the rows kept at one compression event."""
        es = 4 if self.dtype == "f32" else 2
        return 4 * min(self.B, self.L_k) * self.d * es * self.H


# The five configurations (sizes only; values come from the generators below).
CONFIGS = {
    "tiny_f32": Workload("tiny_f32", "f32", H=2, d=64, W=4, n_c=256, B=512, L_k=768, seed=0,
                         sigma=1.0, D=128, eps=0.15, warmup_m=1, n_steps=8),
    "single_step_bf16": Workload("single_step_bf16", "bf16", H=16, d=128, W=4, n_c=6240, B=0,
                                 L_k=24960, seed=1, sigma=0.5),
    "cached_step_bf16": Workload("cached_step_bf16", "bf16", H=24, d=128, W=8, n_c=4680, B=18720,
                                 L_k=23400, seed=2, sigma=0.5, keys="clustered"),
    "streaming_bf16": Workload("streaming_bf16", "bf16", H=24, d=128, W=1, n_c=4680, B=28080,
                               L_k=32760, seed=3, sigma=0.5, keys="ar1", n_steps=4),
    "sweep_bf16": Workload("sweep_bf16", "bf16", H=24, d=128, W=16, n_c=6240, B=37440,
                           L_k=43680, seed=4, sigma=0.5, n_steps=30),
    # The paper's second model family: blocks inside a chunk at staggered noise levels.  A "chunk" of the
    # library is one block here: 5 latent frames of 34 x 60 patches (540P), 12 heads x 128 (hidden 1536); five
    # blocks in flight; the clean region is the 17-frame (5 latent frames) overlap with the previous chunk;
    # thresholds 0.1 / 0.15, four warm-up steps.
    "skyreels_bf16": Workload("skyreels_bf16", "bf16", H=12, d=128, W=5, n_c=10200, B=10200,
                              L_k=20400, seed=5, sigma=0.5, eps=0.1, warmup_m=4, n_steps=50),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller copy of a configuration (for cases the oracle finishes quickly)."""
    return replace(w, **kw)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def normal(shape, seed, sigma=1.0, dtype=torch.float32) -> torch.Tensor:
    return (torch.randn(shape, generator=_gen(seed), dtype=torch.float32) * sigma).to(dtype)


def clustered_keys(H, L, d, seed, n_centres=512, noise=0.05, dtype=torch.bfloat16):
    """Keys = one of n_centres centres ~ N(0,1) (picked uniformly) + N(0, noise^2)."""
    g = _gen(seed)
    centres = torch.randn((H, n_centres, d), generator=g)
    pick = torch.randint(0, n_centres, (H, L), generator=g)
    k = torch.gather(centres, 1, pick[..., None].expand(H, L, d))
    k = k + noise * torch.randn((H, L, d), generator=g)
    return k.to(dtype)


def ar1_keys(H, n_chunks, n_c, d, seed, rho=0.98, sigma=0.5, dtype=torch.bfloat16):
    """Yield per-chunk keys K_c[p] = rho*K_{c-1}[p] + sqrt(1-rho^2)*N(0,1), scaled by sigma."""
    g = _gen(seed)
    state = torch.randn((H, n_c, d), generator=g)
    for _ in range(n_chunks):
        yield (state * sigma).to(dtype)
        state = rho * state + math.sqrt(1.0 - rho * rho) * torch.randn((H, n_c, d), generator=g)


def qkv(w: Workload, seed_offset=0):
    """Q [H, W*n_c, d]; K, V [H, B + W*n_c, d] laid out as [clean region | window]."""
    s = w.seed * 1000 + seed_offset
    L_phys = w.B + w.window_rows
    Q = normal((w.H, w.window_rows, w.d), s + 1, w.sigma, w.torch_dtype)
    if w.keys == "clustered":
        K = clustered_keys(w.H, L_phys, w.d, s + 2, dtype=w.torch_dtype)
    else:
        K = normal((w.H, L_phys, w.d), s + 2, w.sigma, w.torch_dtype)
    V = normal((w.H, L_phys, w.d), s + 3, w.sigma, w.torch_dtype)
    return Q, K, V


def candidates(w: Workload, seed_offset=0):
    """K_cand, V_cand [H, L_k, d] and Q_obs [H, L_q_obs, d] for one compression event."""
    s = w.seed * 1000 + 100 + seed_offset
    if w.keys == "clustered":
        K = clustered_keys(w.H, w.L_k, w.d, s + 1, dtype=w.torch_dtype)
    else:
        K = normal((w.H, w.L_k, w.d), s + 1, w.sigma, w.torch_dtype)
    V = normal((w.H, w.L_k, w.d), s + 2, w.sigma, w.torch_dtype)
    Q_obs = normal((w.H, w.L_q_obs, w.d), s + 3, w.sigma, w.torch_dtype)
    return Q_obs, K, V


def prefix_layout(w: Workload):
    """Segment table and visibility of the layout [clean region | window chunk 0 | 1 | ...].

    Chunk i sees the first B + (i+1)*n_c logical tokens.  Returns plain int32 arrays:
    q_chunk_row_off [W+1], kv_visible_len [W], seg_logical_off [n_seg+1], seg_phys_off [n_seg].
    """
    q_off = np.arange(w.W + 1, dtype=np.int32) * w.n_c
    vis = (w.B + (np.arange(w.W, dtype=np.int32) + 1) * w.n_c).astype(np.int32)
    seg_log, seg_phys = [0], []
    if w.B > 0:
        seg_phys.append(0)
        seg_log.append(w.B)
    for i in range(w.W):
        seg_phys.append(w.B + i * w.n_c)
        seg_log.append(w.B + (i + 1) * w.n_c)
    return q_off, vis, np.asarray(seg_log, np.int32), np.asarray(seg_phys, np.int32)


def indicator_pair(n_chunks, elems_per_chunk, target_r, seed, dtype=torch.bfloat16, sigma=1.0):
    """prev ~ N(0, sigma^2) and cur = prev * (1 +/- target_r[c]) with random signs, both rounded
    to ``dtype``; in exact arithmetic sum|cur-prev| / sum|prev| equals target_r[c] per chunk."""
    g = _gen(seed)
    prev = torch.randn((n_chunks, elems_per_chunk), generator=g) * sigma
    sign = torch.randint(0, 2, (n_chunks, elems_per_chunk), generator=g).float() * 2 - 1
    r = torch.as_tensor(target_r, dtype=torch.float32).reshape(n_chunks, 1)
    prev_q = prev.to(dtype)
    cur = (prev_q.float() * (1.0 + sign * r)).to(dtype)
    return cur.reshape(-1), prev_q.reshape(-1)


def uniform(shape, seed, lo=0.0, hi=1.0) -> torch.Tensor:
    return torch.rand(shape, generator=_gen(seed)) * (hi - lo) + lo


def sweep_targets(n_steps, n_chunks, seed, kappa_end=0.02):
    """r[s, i] = u[s, i] * kappa_s with u ~ U(0,1) and kappa_s geometric from 1 to kappa_end."""
    u = uniform((n_steps, n_chunks), seed)
    kappa = torch.tensor([kappa_end ** (s / max(n_steps - 1, 1)) for s in range(n_steps)])
    return u * kappa[:, None]


def sample_rows(w: Workload, n_uniform, seed, tile=128, chunks=None):
    """Query rows for sampled parity: first / last row of every chunk, the rows on either side of
    every ``tile`` boundary class (first tile, last full tile, ragged tail), plus ``n_uniform`` distinct
    rows drawn uniformly.  With ``chunks`` (a list of chunk ids) both kinds come from those chunks only."""
    chunks = list(range(w.W)) if chunks is None else [int(c) for c in chunks]
    rows = set()
    for c in chunks:
        base = c * w.n_c
        last_full = (w.n_c // tile) * tile
        for r in (0, 1, tile - 1, tile, last_full - 1, last_full, w.n_c - 2, w.n_c - 1):
            if 0 <= r < w.n_c:
                rows.add(base + r)
    if chunks and n_uniform > 0:
        # distinct rows: a random permutation of the chunks' rows, cut to n_uniform
        pool = len(chunks) * w.n_c
        pick = torch.randperm(pool, generator=_gen(w.seed * 1000 + 900 + seed))[:n_uniform]
        extra = torch.tensor(chunks)[pick // w.n_c] * w.n_c + pick % w.n_c
        rows.update(int(x) for x in extra)
    return np.asarray(sorted(rows), np.int32)


def bits(t: torch.Tensor) -> np.ndarray:
    """CPU tensor -> numpy array the oracle accepts (bf16 as uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    return t.numpy()
