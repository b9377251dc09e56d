"""Seeded synthetic Q/K/V shaped like the paper's Qwen3 prefill workloads.

Input construction only: nothing of the method's arithmetic lives here.  Both the CUDA path and
the CPU checker receive the very same bf16 bit patterns produced by `make_inputs`.

These tensors stand in for the Qwen3-30B-A3B / Qwen3-32B activations on RULER / LongBench prompts
that the paper measures on (Sec. 4.1, 4.3): same head counts, head_dim, context lengths and
block sizes; values follow a clustered-keys-plus-needles recipe that produces mean dilution.

Recipe, for layer/prompt l, query head h, KV head hk, block index i or b (block size B):
  V        : i.i.d. N(0, 1)
  Q        : q_t = s_q * muQ[l, h, i] + eps_t,    muQ, eps ~ N(0, I_d)      (s_q = 0: literal i.i.d.)
  K        : k_t = mu[l, hk, b] + sigma[l, hk] * eps_t,  mu ~ N(0, I_d)
             optional log-normal row scaling  k_t *= exp(sigma_ln * z_t),  z ~ N(0, 1)
  needles  : each key block independently with probability p_needle gets ONE row (uniform position)
             overwritten by nu * sqrt(d) * u, u = unit vector of the token-mean of query block j of one
             query head of that KV group, j uniform in [b, M-1] (so aligned queries see it causally).
Everything is drawn from one torch CPU generator seeded with `seed`, then rounded to bf16.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, asdict

import numpy as np
import torch


@dataclass
class SynthConfig:
    name: str
    L: int = 1            # leading batch = prompts x layers
    N: int = 4096         # tokens
    Hq: int = 1
    Hkv: int = 1
    d: int = 128
    B: int = 64           # block size (queries and keys)
    sigma: float | tuple = 0.3      # key noise; a (lo, hi) tuple draws sigma[l, hk] ~ U[lo, hi]
    p_needle: float = 0.10
    sigma_ln: float = 0.0  # log-normal spread of key row norms
    s_q: float = 1.0       # query-block coherence
    nu: float = 1.5        # needle norm in units of sqrt(d)
    seed: int = 20971
    alpha_base: float = 0.22    # Sec. 4.4 defaults
    alpha_rescue: float = 0.18
    n_sink: int = 1
    n_local: int = 1
    n_recent: int = 1

    @property
    def M(self) -> int:
        return (self.N + self.B - 1) // self.B

    def describe(self) -> dict:
        d = asdict(self)
        d["sigma"] = list(self.sigma) if isinstance(self.sigma, tuple) else self.sigma
        return d


def paper_configs() -> dict:
    """The five workload shapes the build is measured on (names follow the benchmark plan)."""
    return {
        "tiny_iid": SynthConfig("tiny_iid", N=4096, Hq=1, Hkv=1, B=64, sigma=0.3, s_q=0.0, seed=20971),
        "tiny": SynthConfig("tiny", N=4096, Hq=1, Hkv=1, B=64, sigma=0.3, s_q=1.0, seed=20972),
        "q30b_32k": SynthConfig("q30b_32k", N=32768, Hq=32, Hkv=4, B=128, sigma=(0.1, 1.0), seed=20973),
        "q30b_64k": SynthConfig("q30b_64k", N=65536, Hq=32, Hkv=4, B=128, sigma=(0.1, 1.0), p_needle=0.05,
                                sigma_ln=0.5, seed=20974),
        "q30b_128k": SynthConfig("q30b_128k", N=131072, Hq=32, Hkv=4, B=128, sigma=(0.1, 1.0), seed=20975),
        # the Qwen3-32B layer shape, one layer at a time, for the block-size sweep
        "q32b_128k_b64": SynthConfig("q32b_128k_b64", N=131072, Hq=64, Hkv=8, B=64, sigma=(0.1, 1.0), seed=20977),
        "q32b_128k_b128": SynthConfig("q32b_128k_b128", N=131072, Hq=64, Hkv=8, B=128, sigma=(0.1, 1.0), seed=20977),
        "q32b_128k_b256": SynthConfig("q32b_128k_b256", N=131072, Hq=64, Hkv=8, B=256, sigma=(0.1, 1.0), seed=20977),
        "q32b_128k_8l": SynthConfig("q32b_128k_8l", L=8, N=131072, Hq=64, Hkv=8, B=128, sigma=(0.1, 1.0),
                                    seed=20976),
    }


def iter_layers(cfg: SynthConfig):
    """Yields (l, Q_l [N,Hq,d], K_l [N,Hkv,d], V_l [N,Hkv,d]) as bf16 CPU tensors, one layer of the batch at a
    time, in order: the same bits make_inputs returns, without holding all layers on the host at once."""
    L, N, Hq, Hkv, d, B = cfg.L, cfg.N, cfg.Hq, cfg.Hkv, cfg.d, cfg.B
    assert Hq % Hkv == 0
    n_keep = N                       # a length that is not a multiple of B is generated padded, then cut
    M, G = (N + B - 1) // B, Hq // Hkv
    N = M * B
    g = torch.Generator(device="cpu")
    g.manual_seed(cfg.seed)

    def randn(*shape):
        return torch.randn(*shape, generator=g, dtype=torch.float32)

    if isinstance(cfg.sigma, tuple):
        lo, hi = cfg.sigma
        sigma = lo + (hi - lo) * torch.rand(L, Hkv, generator=g)
    else:
        sigma = torch.full((L, Hkv), float(cfg.sigma))

    for l in range(L):
        Vl = randn(N, Hkv, d).to(torch.bfloat16)
        muq = randn(M, 1, Hq, d)
        q = randn(M, B, Hq, d)
        if cfg.s_q != 0.0:
            q += cfg.s_q * muq
        Ql = q.view(N, Hq, d).to(torch.bfloat16)
        del q
        mu = randn(M, 1, Hkv, d)
        k = mu + sigma[l].view(1, 1, Hkv, 1) * randn(M, B, Hkv, d)
        if cfg.sigma_ln > 0.0:
            k *= torch.exp(cfg.sigma_ln * randn(M, B, Hkv, 1))
        # needles
        has = torch.rand(M, Hkv, generator=g) < cfg.p_needle
        pos = torch.randint(0, B, (M, Hkv), generator=g)
        frac = torch.rand(M, Hkv, generator=g)
        which = torch.randint(0, G, (M, Hkv), generator=g)
        bb, hh = torch.nonzero(has, as_tuple=True)
        if bb.numel() > 0:
            jj = bb + torch.floor(frac[bb, hh] * (M - bb).float()).long()
            jj = torch.clamp(jj, max=M - 1)
            qh = hh * G + which[bb, hh]
            qmean = Ql.view(M, B, Hq, d).float().mean(dim=1)          # [M, Hq, d]
            u = qmean[jj, qh]                                         # [n, d]
            u = u / u.norm(dim=1, keepdim=True).clamp_min(1e-12)
            k[bb, pos[bb, hh], hh] = cfg.nu * math.sqrt(d) * u
        Kl = k.view(N, Hkv, d).to(torch.bfloat16)
        del k
        if n_keep != N:
            Ql, Kl, Vl = (t[:n_keep].contiguous() for t in (Ql, Kl, Vl))
        yield l, Ql, Kl, Vl


def make_inputs(cfg: SynthConfig):
    """Returns (Q [L,N,Hq,d], K [L,N,Hkv,d], V [L,N,Hkv,d]) as contiguous bf16 CPU tensors."""
    Q = torch.empty(cfg.L, cfg.N, cfg.Hq, cfg.d, dtype=torch.bfloat16)
    K = torch.empty(cfg.L, cfg.N, cfg.Hkv, cfg.d, dtype=torch.bfloat16)
    V = torch.empty(cfg.L, cfg.N, cfg.Hkv, cfg.d, dtype=torch.bfloat16)
    for l, Ql, Kl, Vl in iter_layers(cfg):
        Q[l], K[l], V[l] = Ql, Kl, Vl
    return Q, K, V


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a bf16/fp32 tensor to a float64 numpy array."""
    return t.detach().cpu().to(torch.float64).numpy()
