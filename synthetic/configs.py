"""The benchmark configurations as data, plus a helper that draws one group.

A *group* is the set of linear maps that share one input activation x, hence
one basis P, one coefficient vector, one residual and one gate decision per
token.  GPT-J's parallel block gives three groups per layer
({q, k, v, fc}, {out}, {proj}); the sequential GPT-2 / OPT blocks give four.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List

import torch

from . import generators as G


@dataclass(frozen=True)
class GroupSpec:
    name: str
    d: int
    d_out: tuple          # output width of each map sharing this input
    k: int
    rank: int             # rank of the true activation subspace
    s: int                # directions the true subspace shares with P
    sigma: float          # isotropic noise scale
    p_outlier: float = 0.0
    p_dtype: str = "bf16"


@dataclass(frozen=True)
class StackSpec:
    name: str
    config_id: int
    n_layers: int
    groups: tuple         # GroupSpec per group of one layer (same for every layer)
    eps: float
    steps: int
    batch: int = 1
    note: str = ""
    # indices i (within a layer) of groups whose successor i+1 sits on a parallel branch of the
    # block: neither reads the other's output (GPT-J: attention output projection | MLP down
    # projection; GPT-2 and OPT blocks are sequential, so none)
    concurrent: tuple = ()

    def concurrent_groups(self):
        """Stack-wide indices of the first group of every independent pair."""
        n = len(self.groups)
        return [layer * n + i for layer in range(self.n_layers) for i in self.concurrent]

    @property
    def n_groups(self) -> int:
        return self.n_layers * len(self.groups)

    def bytes_fast_per_step(self) -> int:
        """bytes(P) + bytes(W_P) over the whole stack (bf16 image)."""
        b = 0
        for g in self.groups:
            sp = 2 if g.p_dtype == "bf16" else 4
            b += g.d * g.k * sp + sum(g.d_out) * g.k * 2
        return b * self.n_layers

    def bytes_w_per_group(self):
        return [sum(g.d_out) * g.d * 2 for g in self.groups]

    def bytes_act_per_token(self) -> int:
        return sum(4 * (g.d + sum(g.d_out)) for g in self.groups) * self.n_layers


def gpt2_groups(k, rank, s, sigma, p_out, sigma_wide=None):
    sw = sigma if sigma_wide is None else sigma_wide
    return (
        GroupSpec("qkv", 768, (2304,), k, rank, s, sigma, p_out),
        GroupSpec("attn_out", 768, (768,), k, rank, s, sigma, p_out),
        GroupSpec("fc", 768, (3072,), k, rank, s, sigma, p_out),
        GroupSpec("proj", 3072, (768,), k, rank, s, sw, p_out),
    )


def gptj_groups(k, rank, s, sigma_4k, sigma_16k, p_out=0.0):
    return (
        GroupSpec("qkv_fc", 4096, (4096, 4096, 4096, 16384), k, rank, s, sigma_4k, p_out),
        GroupSpec("attn_out", 4096, (4096,), k, rank, s, sigma_4k, p_out),
        GroupSpec("proj", 16384, (4096,), k, rank, s, sigma_16k, p_out),
    )


def opt_groups(k, rank, s, sigma_4k, sigma_16k, p_out=0.0):
    return (
        GroupSpec("qkv", 4096, (4096, 4096, 4096), k, rank, s, sigma_4k, p_out),
        GroupSpec("attn_out", 4096, (4096,), k, rank, s, sigma_4k, p_out),
        GroupSpec("fc1", 4096, (16384,), k, rank, s, sigma_4k, p_out),
        GroupSpec("fc2", 16384, (4096,), k, rank, s, sigma_16k, p_out),
    )


def config1() -> StackSpec:
    """Single GPT-2-small c_fc map, literal recipe (fires nearly every token:
    8 of the 48 true directions lie outside P)."""
    g = GroupSpec("c_fc", 768, (3072,), 64, 48, 40, 0.02, 0.05)
    return StackSpec("cfg1_gpt2_cfc", 1, 1, (g,), 0.05, 256, 1,
                     "slow-path correctness / latency case")


def config1_fast() -> StackSpec:
    """Companion of config 1 with the true subspace inside span(P) and small
    noise, so the fast path is exercised at the same shape (~5 % fire)."""
    g = GroupSpec("c_fc", 768, (3072,), 64, 48, 48, 0.005, 0.05)
    return StackSpec("cfg1_fast_gpt2_cfc", 11, 1, (g,), 0.05, 256, 1)


def config2() -> StackSpec:
    return StackSpec("cfg2_gpt2_stack", 2, 12, gpt2_groups(128, 96, 96, 0.02, 0.05),
                     0.05, 512, 1, "L2-resident working set")


# Noise scales found by bisection on the oracle's gate rate over 4096 tokens per input width:
# rho ~ sigma*sqrt(d-k)/||z||, tuned so that ~10 % of tokens have rho >= 0.05.
SIGMA_GPTJ_10 = {4096: 0.010667, 16384: 0.005206}


def config3(gate: str = "10") -> StackSpec:
    """GPT-J-6B-shaped stack, batch-1 decode, k=256, eps=0.05.
    gate: "10" (~10 % of tokens gated, the headline), "0" (sigma/4, none gated),
    "23" (~22.8 %, the paper's model-wide slow fraction at this operating point),
    "100" (sigma*4, all gated)."""
    scale = {"10": 1.0, "0": 0.25, "23": 1.0303, "100": 4.0}[gate]
    s4, s16 = SIGMA_GPTJ_10[4096] * scale, SIGMA_GPTJ_10[16384] * scale
    return StackSpec(f"cfg3_gptj_gate{gate}", 3, 28, gptj_groups(256, 200, 200, s4, s16),
                     0.05, 256, 1, concurrent=(1,))


def config4(k: int, eps: float, sigma_scale: float, steps: int = 64) -> StackSpec:
    """OPT-6.7B-shaped stack; sigma_scale multiplies the noise that puts the
    median rho on eps, sweeping the realised gate rate from 0 to 100 %."""
    rank = int(round(0.78 * k))
    import math
    base4 = eps * math.sqrt(rank) / math.sqrt(4096 - k)
    base16 = eps * math.sqrt(rank) / math.sqrt(16384 - k)
    return StackSpec(f"cfg4_opt_k{k}_eps{eps}_s{sigma_scale}", 4, 32,
                     opt_groups(k, rank, rank, base4 * sigma_scale, base16 * sigma_scale),
                     eps, steps, 1)


def config5(p_outlier: float, batch: int = 64, steps: int = 128) -> StackSpec:
    """Batched decode at GPT-J shapes; inliers sit far below eps (rho ~ 0.01),
    the gate rate is forced by the outlier fraction."""
    s4, s16 = SIGMA_GPTJ_10[4096] * 0.2, SIGMA_GPTJ_10[16384] * 0.2
    return StackSpec(f"cfg5_gptj_b{batch}_p{p_outlier}", 5, 28,
                     gptj_groups(256, 200, 200, s4, s16, p_outlier), 0.05, steps, batch,
                     concurrent=(1,))


def materialize_group(stack: StackSpec, layer: int, gi: int, n_tokens: int, device="cpu",
                      want_w: bool = True, want_x: bool = True) -> dict:
    """Draw W (per map), P and x for group ``gi`` of ``layer``.

    Returns dict(W=[bf16 o x d], P=stored basis, Q=fp64 basis, x=[n_tokens][d]
    fp32, outlier=bool mask).  Seeds depend on (config, layer, group/map,
    purpose) only, so any subset can be re-drawn bit-identically.
    """
    g = stack.groups[gi]
    c = stack.config_id
    out = {}
    q = G.gen_basis(g.d, g.k, G.seed_for(c, layer, gi, "P"), device)
    out["Q"] = q
    out["P"] = G.store_basis(q, g.p_dtype)
    if want_w:
        out["W"] = [
            G.gen_weight(o, g.d, G.seed_for(c, layer, 16 * gi + j + 1000, "W"), device)
            for j, o in enumerate(g.d_out)
        ]
    if want_x:
        pt = G.gen_true_basis(q, g.rank, g.s, G.seed_for(c, layer, gi, "P_true"))
        seeds = {p: G.seed_for(c, layer, gi, p)
                 for p in ("z", "noise", "outlier_mask", "outlier_values")}
        out["x"], out["outlier"] = G.gen_activations(pt, n_tokens, g.sigma, g.p_outlier, seeds)
    return out
