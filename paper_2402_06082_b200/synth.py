"""Seeded synthetic token streams with the structure the SubGen paper reports for LLM caches.

The paper shows (t-SNE figure, Section 3.1) that cached KEYS fall into a modest number of tight
clusters spread over the embedding space while VALUES look unstructured. These generators imitate
that: keys come from a Gaussian mixture per (sequence, KV head), optionally with a fraction of
far outliers or slowly drifting component centres, values are isotropic Gaussians with a per-token
scale, queries are isotropic Gaussians.

This module holds input generation only, none of the method's arithmetic, so that the CPU oracle's
tests and the CUDA library's tests can both draw the same inputs from it. It imports neither.

"Within-cluster sigma" is the TOTAL standard deviation of the offset from the component centre
(noise ~ N(0, sigma^2/d I)), so two members of a component are about sigma*sqrt(2) apart.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Hkv: int
    d: int
    dtype: str                    # "fp32" | "bf16"
    n_prompt: int                 # prompt length (maximum when prompt lengths are drawn)
    n_decode: int
    ncomp: int
    sigma: float
    weights: str                  # "uniform" | "dirichlet"
    value_scale: str              # "one" | "lognormal"
    delta: float
    t: int
    s: int
    window: int
    outlier_frac: float = 0.0
    outlier_radius: float = 3.0
    drift: str = "none"           # "none" | "token" (every centre steps every token) | "emission"
    drift_step: float = 0.0
    varlen: Optional[Tuple[int, int]] = None   # (lo, hi): prompt lengths uniform in [lo, hi]
    philox_seed: int = 0
    data_seed: int = 1000
    m_max: int = 4096
    kc_k: int = 0                 # offline k-center compression: centres kept among the older tokens
    kc_r: int = 0                 # ... and most recent tokens kept beside them

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def units(self):
        return self.B * self.Hkv

    def prompt_lens(self) -> List[int]:
        if self.varlen is None:
            return [self.n_prompt] * self.B
        rng = np.random.default_rng(self.data_seed)
        lo, hi = self.varlen
        return [int(x) for x in rng.integers(lo, hi + 1, self.B)]

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five workloads of the benchmark definition (full size).
CFG1 = Workload("cfg1", B=1, H=1, Hkv=1, d=64, dtype="fp32", n_prompt=0, n_decode=4096, ncomp=16, sigma=0.1,
                weights="uniform", value_scale="one", delta=0.5, t=4, s=256, window=64, data_seed=1001, m_max=256)
CFG2 = Workload("cfg2", B=1, H=32, Hkv=32, d=128, dtype="bf16", n_prompt=16384, n_decode=512, ncomp=256, sigma=0.15,
                weights="dirichlet", value_scale="lognormal", delta=0.6, t=8, s=1024, window=256, data_seed=1002,
                m_max=1024)
CFG3 = Workload("cfg3", B=8, H=32, Hkv=32, d=128, dtype="bf16", n_prompt=32768, n_decode=1024, ncomp=1024, sigma=0.15,
                weights="dirichlet", value_scale="lognormal", delta=0.6, t=8, s=2048, window=512, outlier_frac=0.05,
                data_seed=1003, m_max=4096)
CFG4 = Workload("cfg4", B=1, H=32, Hkv=8, d=128, dtype="bf16", n_prompt=131072, n_decode=256, ncomp=4096, sigma=0.15,
                weights="dirichlet", value_scale="lognormal", delta=0.7, t=16, s=4096, window=1024, drift="token",
                drift_step=0.01, data_seed=1004, m_max=131072)
CFG4B = CFG4.scaled(name="cfg4b", drift="emission", m_max=8192)
CFG5 = Workload("cfg5", B=64, H=32, Hkv=32, d=128, dtype="bf16", n_prompt=65536, n_decode=2048, ncomp=1024, sigma=0.15,
                weights="dirichlet", value_scale="lognormal", delta=0.6, t=8, s=2048, window=512, outlier_frac=0.05,
                varlen=(4096, 65536), data_seed=1005, m_max=6144)
# Shape of the paper's end-to-end experiment (Section 3.2, longest context): a 7B Llama-type model has 32 layers
# of 32 heads with d = 128, i.e. 1024 independent (layer, head) caches of one 9k-token context, held here as
# 32 "sequences" of 32 KV heads; the budget r + k is half the context.
KC9K = Workload("kc9k", B=32, H=32, Hkv=32, d=128, dtype="bf16", n_prompt=9000, n_decode=64, ncomp=256, sigma=0.15,
                weights="dirichlet", value_scale="lognormal", delta=0.6, t=8, s=1024, window=512, data_seed=1006,
                m_max=4096, kc_k=3988, kc_r=512)
CONFIGS = {w.name: w for w in (CFG1, CFG2, CFG3, CFG4, CFG4B, CFG5, KC9K)}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _segmented_cumsum(inc: torch.Tensor, comp: torch.Tensor) -> torch.Tensor:
    """inc [U, n, d], comp [U, n] -> running sum of inc over this and the earlier tokens of the same component."""
    U, n, d = inc.shape
    pos = torch.arange(n, device=inc.device).expand(U, n)
    order = torch.argsort(comp * n + pos, dim=1)
    comp_s = torch.gather(comp, 1, order)
    inc_s = torch.gather(inc, 1, order.unsqueeze(-1).expand(U, n, d))
    cs = torch.cumsum(inc_s, dim=1)
    start = torch.ones(U, n, dtype=torch.bool, device=inc.device)
    start[:, 1:] = comp_s[:, 1:] != comp_s[:, :-1]
    start_idx = torch.where(start, pos, torch.zeros_like(pos))
    start_idx = torch.cummax(start_idx, dim=1).values
    before = torch.gather(cs - inc_s, 1, start_idx.unsqueeze(-1).expand(U, n, d))   # cumsum before segment start
    walk_s = cs - before
    walk = torch.empty_like(walk_s)
    walk.scatter_(1, order.unsqueeze(-1).expand(U, n, d), walk_s)
    return walk


def sequence_stream(w: Workload, seq: int, n: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """All tokens of one sequence: K, V [Hkv, n, d] and Q [H, n, d] in the workload's storage dtype.

    The stream is one process: a prompt of length p followed by decode tokens is sequence_stream(...)[:, :p]
    and [:, p:]. Values depend on (data_seed, seq, n), so always ask for the full length once.
    """
    g = _gen(device, w.data_seed * 1000003 + seq)
    U, d = w.Hkv, w.d
    f32 = dict(dtype=torch.float32, device=device)
    cent = torch.randn(U, w.ncomp, d, generator=g, **f32)
    if w.weights == "uniform":
        pi = torch.full((U, w.ncomp), 1.0 / w.ncomp, **f32)
    else:
        e = -torch.log(torch.rand(U, w.ncomp, generator=g, **f32).clamp_min(1e-12))   # Dirichlet(1)
        pi = e / e.sum(dim=1, keepdim=True)
    comp = torch.multinomial(pi, n, replacement=True, generator=g)                    # [U, n]
    K = torch.gather(cent, 1, comp.unsqueeze(-1).expand(U, n, d))
    K = K + (w.sigma / math.sqrt(d)) * torch.randn(U, n, d, generator=g, **f32)
    if w.drift != "none":
        inc = (w.drift_step / math.sqrt(d)) * torch.randn(U, n, d, generator=g, **f32)
        if w.drift == "token":
            # every centre takes one step per token; only the sum of the steps between two emissions
            # of a component is ever observed, and that sum is N(0, gap * step^2/d I)
            pos = torch.arange(n, device=device).expand(U, n)
            order = torch.argsort(comp * n + pos, dim=1)
            comp_s = torch.gather(comp, 1, order)
            pos_s = torch.gather(pos, 1, order)
            gap_s = torch.empty_like(pos_s)
            gap_s[:, 0] = pos_s[:, 0] + 1
            same = comp_s[:, 1:] == comp_s[:, :-1]
            gap_s[:, 1:] = torch.where(same, pos_s[:, 1:] - pos_s[:, :-1], pos_s[:, 1:] + 1)
            gap = torch.empty_like(gap_s)
            gap.scatter_(1, order, gap_s)
            inc = inc * gap.to(torch.float32).sqrt().unsqueeze(-1)
        K = K + _segmented_cumsum(inc, comp)
    if w.outlier_frac > 0:
        o = torch.rand(U, n, generator=g, **f32) < w.outlier_frac
        gdir = torch.randn(U, n, d, generator=g, **f32)
        gdir = w.outlier_radius * gdir / gdir.norm(dim=-1, keepdim=True)
        K = torch.where(o.unsqueeze(-1), gdir, K)
    V = torch.randn(U, n, d, generator=g, **f32)
    if w.value_scale == "lognormal":
        V = V * torch.exp(0.5 * torch.randn(U, n, 1, generator=g, **f32))
    Q = torch.randn(w.H, n, d, generator=g, **f32)
    dt = w.torch_dtype
    return K.to(dt).contiguous(), V.to(dt).contiguous(), Q.to(dt).contiguous()


def batch_stream(w: Workload, n: int, device="cpu"):
    """K, V [B, Hkv, n, d] and Q [B, H, n, d] for all sequences, each of length n."""
    Ks, Vs, Qs = zip(*(sequence_stream(w, b, n, device) for b in range(w.B)))
    return torch.stack(Ks), torch.stack(Vs), torch.stack(Qs)


def to_f32_numpy(x: torch.Tensor) -> np.ndarray:
    """Exact widening of stored values (bf16 or fp32) to a binary32 numpy array on the host."""
    return x.detach().to("cpu", torch.float32).contiguous().numpy()
