"""Seeded synthetic inputs for the sampled linear backward.

This module only draws random tensors; it contains none of the method's arithmetic, so it
can serve both the CUDA library's callers and the CPU checker without coupling them.

The tensors stand in for the transformer layers the paper fine-tunes and pre-trains
(BERT-base / BERT-large / ViT-base shapes and an LLM-sized MLP): layer input X ~ N(0, 1),
weight W ~ N(0, 0.02^2), and an output gradient dY whose rows are Gaussian directions
scaled per datum by lognormal(0, sigma_A) and per token by lognormal(0, sigma_B) -- the
few-heavy-data structure of the per-datum gradient norms shown in the paper's Fig. 3.
Values are rounded once to the storage dtype; everything downstream reads those bytes.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class LayerCase:
    name: str
    N: int
    T: int
    d_in: int
    d_out: int
    dtype: torch.dtype
    sigma_A: float
    sigma_B: float
    rho: float
    nu: float
    data_seed: int = 1234
    zero_fraction: float = 0.0   # share of data whose dY is exactly zero (dropped upstream)

    @property
    def R(self) -> int:
        return self.N * self.T


# The five workloads (shapes and ratios as configured for this repository's benchmark).
CASES = {
    "fp32_small": LayerCase("fp32_small", 4, 64, 256, 256, torch.float32, 1.0, 0.5, 0.5, 0.5),
    "bert_base_ffn_up": LayerCase("bert_base_ffn_up", 32, 128, 768, 3072, torch.bfloat16, 1.5, 1.0, 0.3, 0.4),
    "vit_base_mlp_fc2": LayerCase("vit_base_mlp_fc2", 64, 197, 3072, 768, torch.bfloat16, 1.2, 0.0, 0.4, 0.5),
    "vit_base_mlp_fc1": LayerCase("vit_base_mlp_fc1", 64, 197, 768, 3072, torch.bfloat16, 1.2, 0.0, 0.4, 0.5,
                                  zero_fraction=0.6),
    "bert_large_qkv": LayerCase("bert_large_qkv", 32, 512, 1024, 3072, torch.bfloat16, 1.0, 0.5, 0.5, 0.3),
    "bert_large_attn_out": LayerCase("bert_large_attn_out", 32, 512, 1024, 1024, torch.bfloat16, 1.0, 0.5, 0.5, 0.3),
    "bert_large_ffn_up": LayerCase("bert_large_ffn_up", 32, 512, 1024, 4096, torch.bfloat16, 1.0, 0.5, 0.5, 0.3),
    "bert_large_ffn_down": LayerCase("bert_large_ffn_down", 32, 512, 4096, 1024, torch.bfloat16, 1.0, 0.5, 0.5, 0.3),
    "llm_mlp_up": LayerCase("llm_mlp_up", 8, 2048, 4096, 11008, torch.bfloat16, 0.0, 1.0, 0.3, 0.3),
}


def make_layer(case: LayerCase, batch: int = 0, *, N=None, T=None, d_in=None, d_out=None, device="cpu"):
    """Draw (X [R, d_in], dY [R, d_out], W [d_out, d_in]) for `case`, by default on the CPU.

    With a CUDA `device` the same recipe runs on that device's generator (same distributions and seeds, other
    values than the CPU's): for benchmarks that need many large tensors and no host copy of them.

    `batch` selects an independent mini-batch (same W, fresh X and dY), as the probe's
    Monte-Carlo batches need.  Shape overrides give reduced copies of a workload with the
    same value distributions.
    """
    N = case.N if N is None else N
    T = case.T if T is None else T
    d_in = case.d_in if d_in is None else d_in
    d_out = case.d_out if d_out is None else d_out
    R = N * T
    kw = dict(dtype=torch.float32, device=device)
    gw = torch.Generator(device).manual_seed(case.data_seed)
    W = (torch.randn(d_out, d_in, generator=gw, **kw) * 0.02).to(case.dtype)
    gb = torch.Generator(device).manual_seed(case.data_seed * 1000003 + 7919 * (batch + 1))
    X = torch.randn(R, d_in, generator=gb, **kw).to(case.dtype)
    A = torch.exp(case.sigma_A * torch.randn(N, generator=gb, **kw))
    B = torch.exp(case.sigma_B * torch.randn(N, T, generator=gb, **kw))
    if case.zero_fraction > 0.0:
        dead = torch.rand(N, generator=gb, device=device) < case.zero_fraction
        A = torch.where(dead, torch.zeros_like(A), A)
    dY = torch.randn(R, d_out, generator=gb, **kw)
    dY = (dY * (A[:, None] * B).reshape(R, 1)).to(case.dtype)
    return X, dY, W


def make_preactivation(case: LayerCase, batch: int = 0, *, N=None, T=None, width=None, device="cpu"):
    """Pre-activation H ~ N(0, 1) of shape [R, width] saved by a GELU between two linears."""
    N = case.N if N is None else N
    T = case.T if T is None else T
    width = case.d_in if width is None else width
    g = torch.Generator(device).manual_seed(case.data_seed * 7 + 13 * (batch + 1))
    return torch.randn(N * T, width, generator=g, dtype=torch.float32, device=device).to(case.dtype)
