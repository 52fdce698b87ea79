"""Seeded synthetic layers shaped like the paper's LLaMA / ViT workloads.

This module only draws random inputs (weights W and the two activation
streams X-tilde, X) and names the five benchmark configurations.  It holds
none of the method's arithmetic and is the one module that the CPU oracle's
tests and the CUDA path's tests both import, so that each comparison sees
identical arrays.

Layout: activations are produced token-major, ``[tokens, n]`` float32, one
token batch at a time, so that a batch can be regenerated from
``(config, batch index)`` alone and never has to be stored.  Weights are
``[m, n]`` float32 (rows = output channels), as in the paper's row-vector
notation (Section 3.1).

The real calibration data of the paper (Wikitext2 / C4 activations of LLaMA
layers, ImageNet activations of ViTs) is not available; these inputs stand in
for it, taking its shapes, token counts and rough value structure (heavy
tails, outlier channels, gated-MLP sparsity, LayerNorm-ed tokens).
"""
from __future__ import annotations

import dataclasses

import torch


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    m: int                 # output channels (rows of W)
    n: int                 # input neurons (columns of W, order of H)
    batch_tokens: int      # tokens per accumulate call
    n_batches: int
    act: str               # "gauss" | "student" | "gated" | "layernorm"
    outlier_channels: int
    outlier_scale: float
    noise: float           # relative std of X - X~
    w_std: float
    bits: int
    group: int             # 0 = one grid per output channel
    sym: bool
    blocksize: int
    damp: float
    alpha: float
    w_bf16: bool = False   # weights rounded to bf16 before anyone sees them
    seed: int = 0

    @property
    def tokens(self) -> int:
        return self.batch_tokens * self.n_batches


CONFIGS = {
    # single small linear layer
    "cfg1": LayerConfig("cfg1", 128, 128, 512, 1, "gauss", 4, 20.0, 0.05, 0.02,
                        4, 0, False, 32, 0.01, 0.25),
    # LLaMA-7B-shaped attention projection
    "cfg2": LayerConfig("cfg2", 4096, 4096, 8192, 32, "student", 41, 30.0, 0.05, 0.02,
                        4, 128, False, 128, 0.01, 0.25),
    # LLaMA-3-8B-shaped MLP down projection
    "cfg3": LayerConfig("cfg3", 4096, 14336, 8192, 32, "gated", 0, 1.0, 0.05, 0.015,
                        3, 128, False, 128, 0.01, 0.25),
    # ViT-L / EVA-02-shaped MLP fc1: 8 batches of 16 images x 257 tokens
    "cfg4": LayerConfig("cfg4", 4096, 1024, 4112, 8, "layernorm", 2, 50.0, 0.08, 0.02,
                        3, 0, True, 128, 0.10, 0.25),
    # LLaMA-405B-shaped MLP down projection
    "cfg5": LayerConfig("cfg5", 16384, 53248, 4096, 32, "gated", 0, 1.0, 0.05, 0.015,
                        4, 128, False, 128, 0.01, 0.25, w_bf16=True),
}


def scaled(cfg: LayerConfig, **kw) -> LayerConfig:
    """A copy of ``cfg`` with some fields replaced (smaller test variants)."""
    return dataclasses.replace(cfg, **kw)


_STREAM_W, _STREAM_ACT, _STREAM_PERM = 0, 1, 3


def _gen(cfg: LayerConfig, stream: int, index: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((cfg.seed * 1_000_003 + stream) * 1_000_003 + index + 12345)
    return g


def outlier_channels(cfg: LayerConfig) -> torch.Tensor:
    """Indices of the outlier channels: first entries of a seeded permutation
    (drawn on the CPU so that every device sees the same channels)."""
    g = _gen(cfg, _STREAM_PERM, 0, "cpu")
    return torch.randperm(cfg.n, generator=g)[: cfg.outlier_channels]


def make_weight(cfg: LayerConfig, device="cpu", rows: int | None = None) -> torch.Tensor:
    """W ~ N(0, w_std^2), float32 ``[m, n]`` (bf16-representable if w_bf16).
    Rows are drawn in slabs of 1024 so that any prefix can be made cheaply."""
    m = cfg.m if rows is None else min(rows, cfg.m)
    out = torch.empty((m, cfg.n), dtype=torch.float32, device=device)
    for s, r0 in enumerate(range(0, m, 1024)):
        r1 = min(r0 + 1024, m)
        g = _gen(cfg, _STREAM_W, s, device)
        slab = torch.randn((1024, cfg.n), generator=g, device=device, dtype=torch.float32)
        out[r0:r1] = slab[: r1 - r0] * cfg.w_std
    if cfg.w_bf16:
        out = out.to(torch.bfloat16).to(torch.float32)
    return out


def make_batch(cfg: LayerConfig, b: int, device="cpu", tokens: int | None = None):
    """Token batch ``b``: returns ``(X, Xfp)``, each float32 ``[tokens, n]``.

    ``Xfp`` (the paper's X-tilde) is the full-precision model's layer input,
    ``X`` the quantized model's: ``X = Xfp + N(0, (noise * |Xfp|)^2)``
    elementwise, a stand-in for the drift that earlier quantized layers and
    activation quantization cause.
    """
    t = cfg.batch_tokens if tokens is None else tokens
    n = cfg.n
    g = _gen(cfg, _STREAM_ACT, b, device)

    def randn(*shape):
        return torch.randn(shape, generator=g, device=device, dtype=torch.float32)

    if cfg.act == "gauss":
        xfp = randn(t, n)
    elif cfg.act == "student":
        # Student-t, nu = 4: z / sqrt(chi2_4 / 4)
        z = randn(t, n)
        chi2 = torch.zeros((t, n), device=device, dtype=torch.float32)
        for _ in range(4):
            chi2 += randn(t, n) ** 2
        xfp = z / torch.sqrt(chi2 / 4.0)
    elif cfg.act == "gated":
        # SiLU-gated-like: 60 % of the entries near zero, the rest lognormal
        # magnitudes (mu = -1, sigma = 1) with a random sign.
        u = torch.rand((t, n), generator=g, device=device, dtype=torch.float32)
        z = randn(t, n)
        sgn = torch.where(torch.rand((t, n), generator=g, device=device) < 0.5, -1.0, 1.0)
        xfp = torch.where(u < 0.6, 1e-3 * z, sgn * torch.exp(z - 1.0))
    elif cfg.act == "layernorm":
        z = randn(t, n)
        xfp = (z - z.mean(dim=1, keepdim=True)) / z.std(dim=1, keepdim=True)
    else:
        raise ValueError(cfg.act)
    if cfg.outlier_channels:
        ch = outlier_channels(cfg).to(device)
        xfp[:, ch] *= cfg.outlier_scale
    x = xfp + randn(t, n) * (cfg.noise * xfp.abs())
    return x.contiguous(), xfp.contiguous()


def accumulate_flops(cfg: LayerConfig) -> float:
    """Algorithmic flops of the statistics: H is symmetric (n^2 k), dXX^T is not (2 n^2 k)."""
    return 3.0 * cfg.n * cfg.n * cfg.tokens


def describe(cfg: LayerConfig) -> dict:
    return {
        "workload": cfg.name, "m": cfg.m, "n": cfg.n, "tokens": cfg.tokens,
        "batch_tokens": cfg.batch_tokens, "bits": cfg.bits, "group": cfg.group,
        "sym": cfg.sym, "blocksize": cfg.blocksize, "damp": cfg.damp, "alpha": cfg.alpha,
        "act": cfg.act, "w_dtype": "bf16" if cfg.w_bf16 else "fp32",
    }


__all__ = ["LayerConfig", "CONFIGS", "scaled", "make_weight", "make_batch",
           "outlier_channels", "accumulate_flops", "describe"]
