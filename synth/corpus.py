"""Seeded synthetic multi-vector corpora shaped like the paper's workloads.

Recipe (every config): K mixture means mu_k ~ N(0, I_D); the centroids are the
normalised means.  A document token picks a component uniformly, adds
sigma * N(0, I_D) noise to its mean and is L2-normalised; its centroid id is
the generating component and its residual (token minus centroid) is stored as
a uniform b-bit-per-dimension code over [res_lo, res_hi).  Query tokens are
drawn the same way, independently of every document.

Only inputs are made here.  The residual *encoder* lives here because the
index arrays are inputs of both the CPU oracle and the CUDA library; each of
those implements its own *decoder*.

Generation is chunked (fixed chunk size, one RNG stream per chunk and purpose)
so that corpora with hundreds of millions of tokens never materialise their
raw fp32 vectors, and so that the result does not depend on how much memory
the generating device has.  The same (config, seed, device type) always gives
the same arrays; CPU and CUDA generators give different (equally valid) draws.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_CHUNK_TOKENS = 1 << 20

# RNG stream tags
_S_MEANS, _S_LENS, _S_COMP, _S_NOISE, _S_QCOMP, _S_QNOISE, _S_ROT = range(7)


@dataclass(frozen=True)
class CorpusConfig:
    name: str
    n_docs: int
    len_kind: str            # "uniform" | "lognormal" | "fixed"
    len_lo: int
    len_hi: int
    dim: int
    n_centroids: int
    nbits: int
    n_queries: int
    q_len: int
    nprobe: int
    n_prune: int
    k: int
    len_mean: float = 0.0    # target mean of the truncated log-normal
    sigma: float = 0.3
    res_lo: float = -0.25
    res_hi: float = 0.25
    seed: int = 0

    @property
    def code_bytes(self) -> int:
        return self.dim * self.nbits // 8

    def replace(self, **kw) -> "CorpusConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    # 10k docs, ~640k tokens: the CPU oracle finishes in seconds.
    "tiny": CorpusConfig("tiny", 10_000, "uniform", 32, 96, 128, 1_024, 2, 16, 32, 4, 256, 10),
    # 500k docs, ~60M tokens, ~2.2 GB of centroid ids + codes.
    "mid": CorpusConfig("mid", 500_000, "uniform", 40, 200, 128, 65_536, 2, 1_000, 32, 4, 1_024, 10),
    # passage-corpus-shaped: 8.8M docs, ~600M tokens, ~21.6 GB.
    "large": CorpusConfig("large", 8_800_000, "lognormal", 8, 180, 128, 262_144, 2, 2_000, 32, 4, 4_096, 100,
                          len_mean=68.0),
    # long documents, precision variants (dim x bits).
    "long_d128_b2": CorpusConfig("long_d128_b2", 200_000, "fixed", 512, 512, 128, 32_768, 2, 256, 64, 8, 2_048, 50),
    "long_d128_b1": CorpusConfig("long_d128_b1", 200_000, "fixed", 512, 512, 128, 32_768, 1, 256, 64, 8, 2_048, 50),
    "long_d96_b2": CorpusConfig("long_d96_b2", 200_000, "fixed", 512, 512, 96, 32_768, 2, 256, 64, 8, 2_048, 50),
    "long_d96_b1": CorpusConfig("long_d96_b1", 200_000, "fixed", 512, 512, 96, 32_768, 1, 256, 64, 8, 2_048, 50),
}


@dataclass
class Corpus:
    cfg: CorpusConfig
    centroids: torch.Tensor      # [K, D] float32, unit rows
    cids: torch.Tensor           # [T] int32, document-major
    codes: torch.Tensor          # [T, D*nbits/8] uint8, document-major
    doclens: torch.Tensor        # [N] int32
    raw: Optional[torch.Tensor] = None   # [T, D] float32 uncompressed tokens (small corpora only)
    # RaBitQ 1-bit codes of the (unit-norm) tokens, when requested
    rotation: Optional[torch.Tensor] = None   # [D, D] float32 random orthonormal matrix P
    rq_bits: Optional[torch.Tensor] = None    # [T, D/8] uint8: bit t of byte g = (P o)[8g+t] > 0
    rq_inv_dot: Optional[torch.Tensor] = None  # [T] float32: 1 / <o_p, o_p-bar> = sqrt(D) / sum_x |(P o)[x]|

    @property
    def n_tokens(self) -> int:
        return int(self.cids.numel())


def _gen(seed: int, stream: int, index: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    # distinct, reproducible 63-bit seed per (seed, stream, index)
    s = (seed * 0x9E3779B97F4A7C15 + stream * 0xBF58476D1CE4E5B9 + index * 0x94D049BB133111EB + 0x2545F4914F6CDD1D)
    g.manual_seed(s & 0x7FFFFFFFFFFFFFFF)
    return g


def _lognormal_mu(target_mean: float, sd: float, lo: int, hi: int) -> float:
    """mu such that round(exp(N(mu, sd^2))) truncated to [lo, hi] has the target mean."""
    z = np.linspace(-8.0, 8.0, 200_001)
    w = np.exp(-0.5 * z * z)

    def trunc_mean(mu: float) -> float:
        v = np.rint(np.exp(mu + sd * z))
        keep = (v >= lo) & (v <= hi)
        return float((v * w * keep).sum() / (w * keep).sum())

    a, b = math.log(lo), math.log(hi)
    for _ in range(60):
        m = 0.5 * (a + b)
        if trunc_mean(m) < target_mean:
            a = m
        else:
            b = m
    return 0.5 * (a + b)


def doc_lengths(cfg: CorpusConfig) -> torch.Tensor:
    """[N] int32 token counts (always generated on the CPU: cheap, and the same everywhere)."""
    n = cfg.n_docs
    if cfg.len_kind == "fixed":
        return torch.full((n,), cfg.len_lo, dtype=torch.int32)
    g = _gen(cfg.seed, _S_LENS, 0, "cpu")
    if cfg.len_kind == "uniform":
        return torch.randint(cfg.len_lo, cfg.len_hi + 1, (n,), generator=g, dtype=torch.int32)
    if cfg.len_kind == "lognormal":
        sd = 0.5
        mu = _lognormal_mu(cfg.len_mean, sd, cfg.len_lo, cfg.len_hi)
        out = torch.empty(n, dtype=torch.int32)
        todo = torch.arange(n)
        while todo.numel():
            v = torch.round(torch.exp(mu + sd * torch.randn(todo.numel(), generator=g))).to(torch.int64)
            ok = (v >= cfg.len_lo) & (v <= cfg.len_hi)
            out[todo[ok]] = v[ok].to(torch.int32)
            todo = todo[~ok]
        return out
    raise ValueError(cfg.len_kind)


def mixture_means(cfg: CorpusConfig, device="cpu") -> torch.Tensor:
    g = _gen(cfg.seed, _S_MEANS, 0, device)
    return torch.randn(cfg.n_centroids, cfg.dim, generator=g, device=device, dtype=torch.float32)


def encode_residual(r: torch.Tensor, nbits: int, lo: float, hi: float) -> torch.Tensor:
    """Uniform b-bit bucket index per dimension, packed little-endian within each byte.

    2-bit: dimension 4g+t sits in bits [2t, 2t+1] of byte g; 1-bit: dimension 8g+t in bit t of byte g.
    """
    levels = 1 << nbits
    delta = (hi - lo) / levels
    u = torch.clamp(torch.floor((r - lo) / delta), 0, levels - 1).to(torch.int32)
    per_byte = 8 // nbits
    n, d = u.shape
    u = u.view(n, d // per_byte, per_byte)
    shifts = (torch.arange(per_byte, device=u.device, dtype=torch.int32) * nbits).view(1, 1, per_byte)
    return (u << shifts).sum(dim=2).to(torch.uint8)


def random_rotation(cfg: CorpusConfig) -> torch.Tensor:
    """[D, D] float32 random orthonormal matrix (QR of a Gaussian matrix, on the CPU in float64)."""
    g = _gen(cfg.seed, _S_ROT, 0, "cpu")
    a = torch.randn(cfg.dim, cfg.dim, generator=g, dtype=torch.float64)
    qmat, r = torch.linalg.qr(a)
    qmat = qmat * torch.sign(torch.diagonal(r))[None, :]
    return qmat.to(torch.float32).contiguous()


def encode_rabitq_1bit(x: torch.Tensor, rotation: torch.Tensor):
    """RaBitQ with B = 1 on unit-norm rows x: rotate, keep the signs, and store 1 / <o_p, o_p-bar> where o_p-bar is
    the nearest codeword (sign(o_p) / sqrt(D)).  Returns (bits [n, D/8] uint8, inv_dot [n] float32)."""
    op = x @ rotation.t()
    bits = (op > 0).to(torch.int32)
    n, d = bits.shape
    shifts = torch.arange(8, device=x.device, dtype=torch.int32).view(1, 1, 8)
    packed = (bits.view(n, d // 8, 8) << shifts).sum(dim=2).to(torch.uint8)
    inv_dot = (math.sqrt(d) / op.abs().sum(dim=1)).to(torch.float32)
    return packed, inv_dot


def make_corpus(cfg: CorpusConfig, device="cpu", out_device=None, keep_raw: bool = False,
                rabitq: bool = False) -> Corpus:
    """Generate the index arrays of `cfg` on `device`; results are moved to `out_device` (default: `device`).
    rabitq=True also produces RaBitQ 1-bit codes of the tokens (rotation, rq_bits, rq_inv_dot)."""
    device = torch.device(device)
    out_device = torch.device(out_device) if out_device is not None else device
    assert cfg.dim % 8 == 0 and cfg.nbits in (1, 2)
    doclens = doc_lengths(cfg)
    T = int(doclens.to(torch.int64).sum())
    mu = mixture_means(cfg, device)
    cent = mu / mu.norm(dim=1, keepdim=True)
    cids = torch.empty(T, dtype=torch.int32, device=out_device)
    codes = torch.empty(T, cfg.code_bytes, dtype=torch.uint8, device=out_device)
    raw = torch.empty(T, cfg.dim, dtype=torch.float32, device=out_device) if keep_raw else None
    rot = random_rotation(cfg).to(device) if rabitq else None
    rq_bits = torch.empty(T, cfg.dim // 8, dtype=torch.uint8, device=out_device) if rabitq else None
    rq_inv = torch.empty(T, dtype=torch.float32, device=out_device) if rabitq else None
    for ci, t0 in enumerate(range(0, T, _CHUNK_TOKENS)):
        n = min(_CHUNK_TOKENS, T - t0)
        comp = torch.randint(0, cfg.n_centroids, (n,), generator=_gen(cfg.seed, _S_COMP, ci, device), device=device)
        eps = torch.randn(n, cfg.dim, generator=_gen(cfg.seed, _S_NOISE, ci, device), device=device,
                          dtype=torch.float32)
        x = mu[comp] + cfg.sigma * eps
        x = x / x.norm(dim=1, keepdim=True)
        r = x - cent[comp]
        cids[t0:t0 + n] = comp.to(torch.int32).to(out_device)
        codes[t0:t0 + n] = encode_residual(r, cfg.nbits, cfg.res_lo, cfg.res_hi).to(out_device)
        if keep_raw:
            raw[t0:t0 + n] = x.to(out_device)
        if rabitq:
            b, f = encode_rabitq_1bit(x, rot)
            rq_bits[t0:t0 + n] = b.to(out_device)
            rq_inv[t0:t0 + n] = f.to(out_device)
    return Corpus(cfg, cent.to(out_device).contiguous(), cids, codes, doclens.to(out_device), raw,
                  rot.to(out_device) if rabitq else None, rq_bits, rq_inv)


def make_queries(cfg: CorpusConfig, n_queries: Optional[int] = None, device="cpu", out_device=None) -> torch.Tensor:
    """[n_queries, q_len, D] float32 unit-norm query tokens from the same mixture as the corpus."""
    device = torch.device(device)
    out_device = torch.device(out_device) if out_device is not None else device
    want = cfg.n_queries if n_queries is None else n_queries
    nq = max(want, cfg.n_queries)      # always draw the config's full set, so a prefix is the same queries
    mu = mixture_means(cfg, device)
    n = nq * cfg.q_len
    comp = torch.randint(0, cfg.n_centroids, (n,), generator=_gen(cfg.seed, _S_QCOMP, 0, device), device=device)
    eps = torch.randn(n, cfg.dim, generator=_gen(cfg.seed, _S_QNOISE, 0, device), device=device, dtype=torch.float32)
    x = mu[comp] + cfg.sigma * eps
    x = x / x.norm(dim=1, keepdim=True)
    return x.view(nq, cfg.q_len, cfg.dim)[:want].to(out_device).contiguous()
