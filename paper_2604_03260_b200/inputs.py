"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors; it holds none of the method's arithmetic (no scoring, no
masking, no attention) and is the one piece the CUDA path's callers and the CPU oracle's callers
share.  The paper measured on trained models over text corpora; those are not available, so
these draws stand in for them:

* Q/K/V: i.i.d. N(0,1) drawn in fp32 and rounded to bf16 (round to nearest even).
* centroids: fp32 N(0,1) rows of shape [Hkv, K, D], each normalised to unit length.
* ``clustered`` workloads: one latent label z_i per token from a skewed categorical; every query
  head vector and every key head vector of token i is 2.0 * c[kv(h), z_i] + N(0, I); V stays N(0,1).
* ``runs`` workloads (memberships coherent over positions, as a trained router gives for text whose
  topic persists): the sequence is cut into runs of geometric length (mean ``runs`` tokens); a run draws
  ``topk`` distinct latent groups, a token keeps its run's groups except with probability ``flip``
  (then it draws its own); every query and key head vector of the token is
  ``signal`` * (sum of the centroids of its latent groups) + N(0, I).  Whole 128-token tiles then
  hold one set of groups, so far tiles die or need no mask at all.

Draw order with one ``torch.Generator`` seeded by ``Workload.seed``: centroids, (z), then per head
Q rows, per KV head K rows, per KV head V rows.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    Hq: int
    Hkv: int
    D: int
    n: int
    K: int
    topk: int
    window: int
    softcap: float = 0.0
    scale: float = 0.0          # 0 -> 1/sqrt(D)
    clustered: bool = False
    seed: int = 0
    runs: float = 0.0           # > 0: run-structured latent groups, mean run length in tokens
    flip: float = 0.0           # probability that a token leaves its run's groups
    signal: float = 5.0         # amplitude of the latent centroids in a run-structured draw

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def logit_scale(self) -> float:
        return self.scale if self.scale > 0 else 1.0 / float(np.sqrt(self.D))

    def dense_pairs(self) -> int:
        return self.Hq * self.n * (self.n + 1) // 2

    def with_n(self, n: int, name: str | None = None) -> "Workload":
        return replace(self, n=n, name=name or f"{self.name}@n={n}")


SKEW = (0.4, 0.2, 0.1, 0.1, 0.05, 0.05, 0.05, 0.05)

#: the five parity configurations and the 128K metric point
WORKLOADS = {
    "cfg1": Workload("cfg1-gpt2-124m", 12, 12, 64, 1024, 4, 2, 64, seed=1001),
    "cfg2": Workload("cfg2-llama3-8b", 32, 8, 128, 8192, 4, 2, 512, seed=1002),
    "cfg3": Workload("cfg3-mistral-7b-clustered", 32, 8, 128, 32768, 8, 2, 1024, clustered=True, seed=1003),
    "cfg4": Workload("cfg4-gemma2-9b-softcap", 16, 8, 256, 65536, 4, 1, 4096, softcap=50.0, seed=1004),
    "cfg5": Workload("cfg5-llama3-8b-1m", 32, 8, 128, 1048576, 4, 2, 2048, seed=1005),
    "M128k": Workload("M-llama3-8b-128k", 32, 8, 128, 131072, 4, 2, 2048, seed=1006),
    # the metric point's shape with memberships coherent over positions (runs of ~512 tokens, 0.1 % stray tokens)
    "Mruns": Workload("M-llama3-8b-128k-runs", 32, 8, 128, 131072, 4, 2, 2048, seed=1007, runs=512.0, flip=0.001),
    "Mruns1": Workload("M-llama3-8b-128k-runs-top1", 32, 8, 128, 131072, 4, 1, 2048, seed=1008, runs=512.0, flip=0.001),
}


def _randn_bf16(shape, gen, device, mean=None):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if mean is not None:
        x += mean
    return x.to(torch.bfloat16)


def make_inputs(wl: Workload, device: str = "cpu"):
    """Draw (Q [Hq,n,D] bf16, K [Hkv,n,D] bf16, V [Hkv,n,D] bf16, C [Hkv,K,D] fp32) on ``device``.

    The values depend on the device of the generator (CPU and CUDA generators differ); a test or a
    bench run draws once and hands the same tensors to both sides.
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(wl.seed)
    C = torch.randn((wl.Hkv, wl.K, wl.D), generator=gen, device=device, dtype=torch.float32)
    C = C / C.norm(dim=-1, keepdim=True)
    z = None
    member = None               # runs: [n, K] 0/1 latent memberships
    if wl.clustered:
        p = torch.tensor(SKEW[: wl.K], dtype=torch.float32, device=device)
        p = p / p.sum()
        z = torch.multinomial(p, wl.n, replacement=True, generator=gen)
    elif wl.runs > 0:
        start = torch.rand(wl.n, generator=gen, device=device) < 1.0 / wl.runs
        run = torch.cumsum(start.to(torch.int64), 0)                          # run index of every token
        nrun = int(run[-1].item()) + 1
        # a random subset of topk groups per run and per token: the topk smallest of K uniform draws
        pick = lambda rows: (torch.rand((rows, wl.K), generator=gen, device=device).argsort(dim=1) < wl.topk)
        of_run, own = pick(nrun), pick(wl.n)
        stray = torch.rand(wl.n, generator=gen, device=device) < wl.flip
        member = torch.where(stray[:, None], own, of_run[run]).to(torch.float32)
    Q = torch.empty((wl.Hq, wl.n, wl.D), dtype=torch.bfloat16, device=device)
    K = torch.empty((wl.Hkv, wl.n, wl.D), dtype=torch.bfloat16, device=device)
    V = torch.empty((wl.Hkv, wl.n, wl.D), dtype=torch.bfloat16, device=device)
    def mean_of(hk):
        if z is not None:
            return 2.0 * C[hk][z]
        if member is not None:
            return wl.signal * (member @ C[hk])
        return None
    for h in range(wl.Hq):
        Q[h] = _randn_bf16((wl.n, wl.D), gen, device, mean_of(h // wl.G))
    for hk in range(wl.Hkv):
        K[hk] = _randn_bf16((wl.n, wl.D), gen, device, mean_of(hk))
    for hk in range(wl.Hkv):
        V[hk] = _randn_bf16((wl.n, wl.D), gen, device)
    return Q, K, V, C


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array of its bit patterns (on the host)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def sample_rows(wl: Workload, per_head: int, seed: int | None = None, tile: int = 128) -> np.ndarray:
    """Rows to check on workloads too large for an all-rows comparison: ``per_head`` seeded draws
    per query head plus boundary rows (first rows, both sides of the window edge and of a tile
    edge, the middle, the last tile, the last row).  Returns int64 [R, 2] of (head, token)."""
    rng = np.random.default_rng(wl.seed * 7919 + 13 if seed is None else seed)
    n, w = wl.n, wl.window
    forced = [0, 1, w - 1, w, w + 1, tile - 1, tile, tile + 1, n // 2, n - tile, n - 2, n - 1]
    forced = sorted({int(r) for r in forced if 0 <= r < n})
    rows = []
    for h in range(wl.Hq):
        draw = rng.integers(0, n, size=max(0, per_head - len(forced)))
        for i in forced + [int(x) for x in draw]:
            rows.append((h, i))
    return np.asarray(rows, dtype=np.int64)
