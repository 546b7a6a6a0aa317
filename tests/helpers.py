"""Shared test plumbing: torch <-> oracle conversions, tolerance checks, scenario builders.

The scenario builders only draw inputs (through ``workloads``) and hand the same
tensors to the oracle (as numpy bit patterns) and to the CUDA library (as device
tensors).  Nothing flows from the CUDA library into the oracle.
"""
import numpy as np
import torch

import paper_2609_34060_b200 as kvc
from paper_2609_34060_b200 import workloads as wl
from oracle import kvc_oracle as orc

BF16_REL = 2.0 ** -7     # |err| <= 2^-7 |ref| + 1e-3 for bf16 results
BF16_ABS = 1e-3


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def oracle_cache(c: "kvc.Cache") -> orc.Cache:
    if c.page_table is None:
        return orc.Cache(bits_of(c.k), bits_of(c.v))
    return orc.Cache(bits_of(c.k), bits_of(c.v), T=c.T, page_table=c.page_table.cpu().numpy())


def oracle_state(s: "kvc.State") -> orc.State:
    if s.r == 0 or s.n_cov == 0:
        z = np.zeros((1, 1, 0, 0), np.float32)
        return orc.State(z, z, z, z, n_cov=0)
    f = lambda t: t.detach().cpu().to(torch.float32).numpy()
    return orc.State(f(s.coeff_k), f(s.coeff_v), f(s.basis_k), f(s.basis_v), n_cov=s.n_cov)


def logical_bits(c, which):
    """[L,H,T,d] uint16 in logical token order, from a kvc.Cache or an orc.Cache."""
    oc = c if isinstance(c, orc.Cache) else oracle_cache(c)
    return np.stack([np.stack([oc.get_bits(which, l, h) for h in range(oc.H)]) for l in range(oc.L)])


def tol_ratio(got_bits: np.ndarray, ref: np.ndarray) -> float:
    """max over elements of |got - ref| / (2^-7 |ref| + 1e-3); must be <= 1."""
    got = orc.bf16_to_f64(got_bits)
    err = np.abs(got - ref)
    tol = BF16_REL * np.abs(ref) + BF16_ABS
    return float(np.max(err / tol)) if err.size else 0.0


def ulp_mismatch_fraction(got_bits, exp_bits) -> float:
    """Fraction of elements whose bf16 pattern differs from the oracle's rounding."""
    return float(np.mean(got_bits != exp_bits)) if got_bits.size else 0.0


def to_dev(c_cpu: "kvc.Cache", dev) -> "kvc.Cache":
    pt = None if c_cpu.page_table is None else c_cpu.page_table.to(dev)
    return kvc.Cache(c_cpu.k.to(dev), c_cpu.v.to(dev), T=c_cpu.T if pt is not None else None, page_table=pt)


def state_to_dev(s: "kvc.State", dev) -> "kvc.State":
    mv = lambda t: None if t is None else t.to(dev)
    return kvc.State(mv(s.coeff_k), mv(s.coeff_v), mv(s.basis_k), mv(s.basis_v), n_cov=s.n_cov,
                     grouping=getattr(s, "grouping", kvc.KVC_GROUP_HEAD))


def make_cache(cfg: wl.Config, table_tag=0, extra_pages=3):
    """Agent 0's cache on the CPU as a kvc.Cache (contiguous or paged per cfg)."""
    if not cfg.paged:
        k, v = wl.base_cache(cfg, "cpu")
        return kvc.Cache(k, v)
    npg = wl.n_pages(cfg.T, cfg.page)
    P = npg + extra_pages
    pt = wl.page_table(npg, P, cfg.seed, table_tag)
    k, v = wl.base_cache(cfg, "cpu", table=pt, n_phys=P)
    return kvc.Cache(k, v, T=cfg.T, page_table=pt)


def make_state(cfg: wl.Config, hop: int, n_cov=None, r=None, basis_dtype=torch.float32) -> "kvc.State":
    s = wl.hop_state(cfg, hop, "cpu", r=r)
    n = cfg.T if n_cov is None else n_cov
    return kvc.State(s["coeff_k"][:, :, :n].contiguous(), s["coeff_v"][:, :, :n].contiguous(),
                     s["basis_k"].to(basis_dtype), s["basis_v"].to(basis_dtype), n_cov=n)


def empty_dst(src_cpu: "kvc.Cache", cfg: wl.Config, dev, table_tag=50, fill=None):
    """A device destination with the source's geometry; paged ones get their own table."""
    if src_cpu.page_table is None:
        d = src_cpu.empty_like(fill=fill)
        return kvc.Cache(d.k.to(dev), d.v.to(dev))
    pt = wl.page_table(src_cpu.page_table.numel(), src_cpu.P, cfg.seed, table_tag)
    d = src_cpu.empty_like(page_table=pt, fill=fill)
    return kvc.Cache(d.k.to(dev), d.v.to(dev), T=src_cpu.T, page_table=pt.to(dev))


def inv_freq(cfg: wl.Config):
    return orc.rope_inv_freq(cfg.d, cfg.theta)
