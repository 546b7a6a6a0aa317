"""Seeded synthetic inputs for the KV-correction hot path.

This module only *draws* inputs: Gaussian caches with the structure of the
benchmark configurations (outlier key channels, image-patch spans), random
coefficients, orthonormal bases (QR of a Gaussian, a library routine), prefix
lengths, shuffled page tables, request mixes.  It holds none of the method's
arithmetic -- no re-alignment, no correction, no projection -- so the CPU
oracle and the CUDA library can both be fed from it without sharing anything
that could hide a common mistake.  Quantities *derived* by the method (a true
target cache = aligned source + low-rank deviation + noise) are produced by
whoever consumes the inputs: the oracle in the tests, the library in the
benchmark.

All tensors are torch tensors on the requested device; bf16 caches are
``torch.bfloat16``.  Every draw uses its own ``torch.Generator`` seeded from
(seed, a small tag), so one tensor can be regenerated without the others.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    L: int
    H: int
    d: int
    T: int                      # shared tokens (single-request configs)
    n_agents: int
    r: int
    theta: float = 500000.0
    paged: bool = False
    page: int = 16
    outliers: int = 0           # outlier key channels per (layer, head), scaled 10x
    image_spans: Sequence = ()  # (start, stop) token ranges with a mean offset
    prefix_lo: int = 64
    prefix_hi: int = 512
    prefix: Optional[Sequence[int]] = None   # fixed prefix lengths, else uniform in [lo, hi]
    sigma: float = 1e-3         # std of the additive noise on a true target
    seed: int = 0

    def scaled(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


_VLM_SPANS = tuple((4096 * s + 512, 4096 * s + 1536) for s in range(4))

CONFIGS = {
    # config 1: parity-sized
    "tiny": Config("tiny", L=2, H=2, d=64, T=256, n_agents=2, r=8, theta=10000.0, prefix=(32, 48)),
    # config 2: the graded throughput workload
    "llama8b_8k": Config("llama8b_8k", L=32, H=8, d=128, T=8192, n_agents=4, r=32, outliers=4),
    # config 3: paged, image-patch spans
    "vlm_16k": Config("vlm_16k", L=28, H=4, d=128, T=16384, n_agents=5, r=32, paged=True,
                      image_spans=_VLM_SPANS),
    # config 5: long context, paged, r = 64
    "llama70b_32k": Config("llama70b_32k", L=80, H=8, d=128, T=32768, n_agents=8, r=64, paged=True,
                           outliers=4),
}


def _gen(device, seed: int, tag: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(tag)) & 0x7FFFFFFFFFFF)
    return g


def prefix_lengths(cfg: Config) -> List[int]:
    """Tokens that precede the shared context in each agent's sequence."""
    if cfg.prefix is not None:
        return [int(p) for p in cfg.prefix]
    g = _gen("cpu", cfg.seed, 1)
    return [int(x) for x in torch.randint(cfg.prefix_lo, cfg.prefix_hi + 1, (cfg.n_agents,), generator=g)]


def page_table(n_logical: int, n_phys: int, seed: int, tag: int, device="cpu") -> torch.Tensor:
    """A shuffled int32 logical->physical page map (distinct physical pages)."""
    assert n_phys >= n_logical
    g = _gen("cpu", seed, 100 + tag)
    perm = torch.randperm(n_phys, generator=g)[:n_logical].to(torch.int32)
    return perm.to(device)


def n_pages(T: int, page: int) -> int:
    return (T + page - 1) // page


def outlier_channels(cfg: Config) -> Optional[torch.Tensor]:
    """[L, H, cfg.outliers] int64 channel indices, drawn once per (layer, head)."""
    if cfg.outliers <= 0:
        return None
    g = _gen("cpu", cfg.seed, 2)
    idx = torch.stack([torch.randperm(cfg.d, generator=g)[: cfg.outliers] for _ in range(cfg.L * cfg.H)])
    return idx.reshape(cfg.L, cfg.H, cfg.outliers)


def base_cache(cfg: Config, device="cpu", table: Optional[torch.Tensor] = None, n_phys: Optional[int] = None):
    """Agent 0's cache.  Contiguous: (K, V) bf16 [L,H,T,d].  Paged: pools bf16
    [L,P,H,page,d] drawn directly in pool order (every physical page holds data)."""
    dev = torch.device(device)
    gk, gv = _gen(dev, cfg.seed, 10), _gen(dev, cfg.seed, 11)
    if not cfg.paged:
        shape = (cfg.L, cfg.H, cfg.T, cfg.d)
    else:
        assert table is not None and n_phys is not None
        shape = (cfg.L, n_phys, cfg.H, cfg.page, cfg.d)
    k = torch.empty(shape, dtype=torch.float32, device=dev).normal_(generator=gk)
    v = torch.empty(shape, dtype=torch.float32, device=dev).normal_(generator=gv)
    oc = outlier_channels(cfg)
    if oc is not None:
        scale = torch.ones(cfg.L, cfg.H, cfg.d)
        scale.scatter_(2, oc, 10.0)
        scale = scale.to(dev)
        if not cfg.paged:
            k *= scale[:, :, None, :]
        else:
            k *= scale[:, None, :, None, :]
    if cfg.image_spans:
        go = _gen("cpu", cfg.seed, 12)
        for (a, b) in cfg.image_spans:
            if a >= cfg.T:
                continue
            b = min(b, cfg.T)
            off_k = (0.5 * torch.randn(cfg.L, cfg.H, cfg.d, generator=go)).to(dev)
            off_v = (0.5 * torch.randn(cfg.L, cfg.H, cfg.d, generator=go)).to(dev)
            if not cfg.paged:
                k[:, :, a:b, :] += off_k[:, :, None, :]
                v[:, :, a:b, :] += off_v[:, :, None, :]
            else:
                assert a % cfg.page == 0
                full = b // cfg.page
                phys = table[a // cfg.page: full].to(torch.int64).to(dev)
                k[:, phys] += off_k[:, None, :, None, :]
                v[:, phys] += off_v[:, None, :, None, :]
                if b % cfg.page:                          # the span ends inside a page
                    last = int(table[full])
                    k[:, last, :, : b % cfg.page] += off_k[:, :, None, :]
                    v[:, last, :, : b % cfg.page] += off_v[:, :, None, :]
    return k.to(torch.bfloat16), v.to(torch.bfloat16)


def orthonormal_basis(L: int, H: int, r: int, d: int, seed: int, tag: int, device="cpu") -> torch.Tensor:
    """fp32 [L,H,r,d] with orthonormal rows: Q^T from the QR of a d x r Gaussian."""
    g = _gen("cpu", seed, 200 + tag)
    a = torch.randn(L, H, d, r, dtype=torch.float64, generator=g)
    q, _ = torch.linalg.qr(a)
    return q.transpose(-1, -2).contiguous().to(torch.float32).to(device)


def coefficients(L: int, H: int, T: int, r: int, seed: int, tag: int, device="cpu", scale: float = 1.0) -> torch.Tensor:
    """fp32 [L,H,T,r] ~ N(0, scale^2)."""
    dev = torch.device(device)
    g = _gen(dev, seed, 300 + tag)
    c = torch.empty((L, H, T, r), dtype=torch.float32, device=dev).normal_(generator=g)
    return c * scale if scale != 1.0 else c


def noise(shape, seed: int, tag: int, device="cpu") -> torch.Tensor:
    """Standard normal fp32 draws; the consumer scales them by cfg.sigma."""
    dev = torch.device(device)
    g = _gen(dev, seed, 400 + tag)
    return torch.empty(shape, dtype=torch.float32, device=dev).normal_(generator=g)


def hop_state(cfg: Config, hop: int, device="cpu", T: Optional[int] = None, r: Optional[int] = None):
    """The true rank-r state of hop ``hop`` (1-based): dict with coeff_k/v, basis_k/v."""
    T = cfg.T if T is None else T
    r = cfg.r if r is None else r
    return {
        "coeff_k": coefficients(cfg.L, cfg.H, T, r, cfg.seed, 4 * hop + 0, device),
        "coeff_v": coefficients(cfg.L, cfg.H, T, r, cfg.seed, 4 * hop + 1, device),
        "basis_k": orthonormal_basis(cfg.L, cfg.H, r, cfg.d, cfg.seed, 4 * hop + 2, device),
        "basis_v": orthonormal_basis(cfg.L, cfg.H, r, cfg.d, cfg.seed, 4 * hop + 3, device),
    }


# --------------------------------------------------------------------------
# config 4: the ragged serving batch
# --------------------------------------------------------------------------


@dataclasses.dataclass(frozen=True)
class Request:
    T: int
    n_agents: int
    r: int
    prefix: tuple


def clustered_rows(T: int, d: int, seed: int, tag: int):
    """A [T, d] bf16 matrix whose singular values come in a few clusters of (nearly) equal values
    over a low floor: orthonormal columns (QR of a Gaussian) times the drawn values times an
    orthogonal matrix, rounded to bf16 (which spreads every cluster by about 2^-9).  Returns the
    matrix and the singular values drawn.  A stress input for the truncated SVD of the update."""
    g = _gen("cpu", seed, tag)
    n_cl = int(torch.randint(1, 6, (1,), generator=g))
    vals: List[float] = []
    for _ in range(n_cl):
        level = 10.0 ** float(torch.empty(1).uniform_(-2.0, 1.0, generator=g))
        vals += [level] * int(torch.randint(1, 12, (1,), generator=g))
    floor = 10.0 ** float(torch.empty(1).uniform_(-5.0, -3.0, generator=g))
    sv = torch.tensor(sorted((vals + [floor] * d)[:d], reverse=True), dtype=torch.float64)
    u, _ = torch.linalg.qr(torch.randn(T, d, generator=g, dtype=torch.float64))
    v, _ = torch.linalg.qr(torch.randn(d, d, generator=g, dtype=torch.float64))
    return ((u * sv) @ v.T * 16.0).to(torch.bfloat16), sv


def serving_batch(n_requests: int = 64, seed: int = 0, median_T: int = 4096, sigma_ln: float = 0.6,
                  t_lo: int = 1024, t_hi: int = 32768, agents_lo: int = 3, agents_hi: int = 6,
                  ranks: Sequence[int] = (16, 32, 64), prefix_lo: int = 64, prefix_hi: int = 512) -> List[Request]:
    """Per-request shared length ~ lognormal(median, sigma_ln) clipped to [t_lo, t_hi]
    (kept ragged: not rounded to the page size), 3-6 agents, rank drawn from ``ranks``."""
    g = _gen("cpu", seed, 500)
    z = torch.randn(n_requests, generator=g, dtype=torch.float64)
    T = torch.clamp(torch.round(torch.exp(math.log(median_T) + sigma_ln * z)), t_lo, t_hi).to(torch.int64)
    na = torch.randint(agents_lo, agents_hi + 1, (n_requests,), generator=g)
    ri = torch.randint(0, len(ranks), (n_requests,), generator=g)
    reqs = []
    for i in range(n_requests):
        pf = torch.randint(prefix_lo, prefix_hi + 1, (int(na[i]),), generator=g)
        reqs.append(Request(int(T[i]), int(na[i]), int(ranks[int(ri[i])]), tuple(int(x) for x in pf)))
    return reqs
