"""Seeded generators for weights, bases and activations.

Everything is drawn with a seeded ``torch.Generator`` on the requested device
(CPU for the small configurations, the GPU for the multi-GB weight sets) and the
same bits are then handed to both the CUDA path and the oracle.  Nothing here
computes a projection, a gate or a layer output.

Recipe (stand-in for the paper's GPT-2 / GPT-J / OPT weights and its 512-token
evaluation text, neither of which is available offline):
  W       iid N(0, 0.02^2), drawn in fp32, rounded to nearest-even bf16, [o][d].
  P       Q factor of the thin QR of a d x k Gaussian in fp64, columns
          sign-normalised so diag(R) > 0; stored as bf16 (default) or fp32.
  P_true  d x rank orthonormal: the first s columns of Q plus rank-s
          orthonormal directions drawn in the orthogonal complement of span(Q).
  x       inlier:  P_true z + sigma n,  z ~ N(0, I_rank), n ~ N(0, I_d), fp64 -> fp32
          outlier: n' sqrt(rank/d), full-rank Gaussian with the same expected
          norm, chosen per token by a seeded Bernoulli(p) mask.
"""
from __future__ import annotations

import numpy as np
import torch

PURPOSE = dict(W=0, P=1, P_true=2, z=3, noise=4, outlier_mask=5, outlier_values=6)


def seed_for(config: int, layer: int, group_or_map: int, purpose: str) -> int:
    return 1_000_003 * config + 10_007 * layer + 101 * group_or_map + PURPOSE[purpose]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gen_weight(o: int, d: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    """[o][d] bf16, iid N(0, std^2) drawn in fp32 then rounded to bf16."""
    w = torch.empty((o, d), dtype=torch.float32, device=device)
    w.normal_(0.0, std, generator=_gen(seed, device))
    return w.to(torch.bfloat16)


def gen_basis(d: int, k: int, seed: int, device="cpu") -> torch.Tensor:
    """Orthonormal d x k basis in fp64 (QR of a seeded Gaussian)."""
    a = torch.empty((d, k), dtype=torch.float64, device=device)
    a.normal_(0.0, 1.0, generator=_gen(seed, device))
    q, r = torch.linalg.qr(a, mode="reduced")
    sign = torch.sign(torch.diagonal(r))
    sign[sign == 0] = 1.0
    return (q * sign).contiguous()   # LAPACK hands back column-major strides


def gen_true_basis(q: torch.Tensor, rank: int, s: int, seed: int) -> torch.Tensor:
    """d x rank orthonormal basis sharing its first s directions with q."""
    d, k = q.shape
    assert 0 <= s <= min(rank, k) and rank <= d
    if s == rank:
        return q[:, :s].contiguous()
    extra = torch.empty((d, rank - s), dtype=torch.float64, device=q.device)
    extra.normal_(0.0, 1.0, generator=_gen(seed, q.device))
    # two sweeps of projection out of span(q), then orthonormalise among themselves
    for _ in range(2):
        extra = extra - q @ (q.T @ extra)
    e, _ = torch.linalg.qr(extra, mode="reduced")
    for _ in range(2):
        e = e - q @ (q.T @ e)
        e, _ = torch.linalg.qr(e, mode="reduced")
    return torch.cat([q[:, :s], e], dim=1).contiguous()


def gen_activations(p_true: torch.Tensor, n_tokens: int, sigma: float, p_outlier: float,
                    seeds: dict):
    """[n_tokens][d] fp32 activations and the outlier mask (bool, on CPU)."""
    d, rank = p_true.shape
    dev = p_true.device
    z = torch.empty((n_tokens, rank), dtype=torch.float64, device=dev)
    z.normal_(0.0, 1.0, generator=_gen(seeds["z"], dev))
    n = torch.empty((n_tokens, d), dtype=torch.float64, device=dev)
    n.normal_(0.0, 1.0, generator=_gen(seeds["noise"], dev))
    x = z @ p_true.T + sigma * n
    mask = torch.zeros(n_tokens, dtype=torch.bool, device=dev)
    if p_outlier > 0.0:
        u = torch.empty(n_tokens, dtype=torch.float64, device=dev)
        u.uniform_(0.0, 1.0, generator=_gen(seeds["outlier_mask"], dev))
        mask = u < p_outlier
        o = torch.empty((n_tokens, d), dtype=torch.float64, device=dev)
        o.normal_(0.0, 1.0, generator=_gen(seeds["outlier_values"], dev))
        o = o * float(np.sqrt(rank / d))
        x = torch.where(mask[:, None], o, x)
    return x.to(torch.float32), mask.cpu()


def store_basis(q: torch.Tensor, dtype: str = "bf16") -> torch.Tensor:
    """Round the fp64 basis to its storage type."""
    q = q.contiguous()
    return (q.to(torch.bfloat16) if dtype == "bf16" else q.to(torch.float32)).contiguous()


def to_bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    """Stored tensor -> the numpy array the oracle takes (uint16 bits or fp32)."""
    if t.dtype == torch.bfloat16:
        return to_bf16_bits(t)
    return t.detach().contiguous().cpu().numpy()
