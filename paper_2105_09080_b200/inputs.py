"""Seeded synthetic inputs shared by the tests of the CUDA path and of the oracle.

This module only draws numbers; it holds none of the method's arithmetic (no
gradient, no mixing, no schedule).  Everything is generated on the host with
numpy's seeded generators so both sides receive bit-identical arrays.

Shapes follow the workloads of the paper's experiments at the sizes the
benchmark configurations name: an n x d fp32 parameter matrix with per-node
quadratic targets b_i (standing in for ResNet-50- and BERT-Large-sized models),
and a per-node logistic-regression data set (Section 5.1 structure).
"""
from __future__ import annotations

import numpy as np


def quadratic_inputs(n: int, d: int, seed: int, x0: str = "zero", x0_std: float = 1.0,
                     b_shift: float = 0.0):
    """Return (X0, B) as float32 arrays of shape (n, d).

    x0: 'zero' | 'shared' (one N(0, x0_std^2) row copied to every node) |
        'per_node' (independent rows).  B_ij ~ N(0,1) + b_shift * s_i with one
        s_i ~ N(0,1) per node.
    """
    rng = np.random.default_rng(seed)
    B = rng.standard_normal((n, d), dtype=np.float32)
    if b_shift != 0.0:
        s = rng.standard_normal((n, 1), dtype=np.float32)
        B = (B + np.float32(b_shift) * s).astype(np.float32)
    if x0 == "zero":
        X0 = np.zeros((n, d), dtype=np.float32)
    elif x0 == "shared":
        row = (np.float32(x0_std) * rng.standard_normal((1, d), dtype=np.float32))
        X0 = np.repeat(row, n, axis=0).astype(np.float32)
    elif x0 == "per_node":
        X0 = (np.float32(x0_std) * rng.standard_normal((n, d), dtype=np.float32)).astype(np.float32)
    else:
        raise ValueError(x0)
    return np.ascontiguousarray(X0), np.ascontiguousarray(B)


def logistic_inputs(n: int, m: int, d: int, seed: int, hetero: float = 0.5,
                    label_noise: float = 0.1):
    """Return (A, y): A float32 (n, m, d) with N(0,1)/sqrt(d) entries, y float32 (n, m) in {-1,+1}.

    Labels are sign(A_i x*_i + label_noise * N(0,1)) with x*_i = x* + hetero * N(0,1),
    x* ~ N(0,1); sign(0) counts as +1.
    """
    rng = np.random.default_rng(seed)
    A = (rng.standard_normal((n, m, d), dtype=np.float32) / np.float32(np.sqrt(d))).astype(np.float32)
    x_star = rng.standard_normal(d)
    y = np.empty((n, m), dtype=np.float32)
    for i in range(n):
        xi = x_star + hetero * rng.standard_normal(d)
        margin = A[i].astype(np.float64) @ xi + label_noise * rng.standard_normal(m)
        y[i] = np.where(margin >= 0.0, 1.0, -1.0)
    return np.ascontiguousarray(A), np.ascontiguousarray(y)


def logistic_inputs_device(n: int, m: int, d: int, seed: int, device="cuda", hetero: float = 0.5,
                           label_noise: float = 0.1):
    """Same recipe as ``logistic_inputs`` drawn on the device with torch's seeded generator
    (a different random stream, hence different numbers): (A, y) as float32 CUDA tensors.
    For workloads too large to ship from the host on every run."""
    import torch
    gen = torch.Generator(device=device).manual_seed(seed)
    A = torch.randn((n, m, d), device=device, generator=gen) / d ** 0.5
    x_star = torch.randn(d, device=device, generator=gen)
    xi = x_star[None, :] + hetero * torch.randn((n, d), device=device, generator=gen)
    margin = torch.einsum("nmd,nd->nm", A, xi) + label_noise * torch.randn((n, m), device=device, generator=gen)
    y = torch.where(margin >= 0, 1.0, -1.0).to(torch.float32).contiguous()
    return A.contiguous(), y


def convex_experiment_inputs(n: int, m: int = 8000, d: int = 10, seed: int = 0, iid: bool = False):
    """Synthetic data of the paper's logistic-regression experiment (Section 5.1): features
    h ~ N(0, 10 I_d); a unit-norm x*_i per node (one shared x* when iid); label +1 with
    probability 1 / (1 + exp(-h^T x*_i)), else -1.  Returns (A, y) float32 with the feature
    dimension zero-padded to a multiple of 4 (padded weights receive zero gradient and stay 0)."""
    rng = np.random.default_rng(seed)
    dp = (d + 3) // 4 * 4
    A = np.zeros((n, m, dp), dtype=np.float32)
    A[:, :, :d] = rng.normal(0.0, np.sqrt(10.0), size=(n, m, d)).astype(np.float32)
    shared = rng.standard_normal(d)
    y = np.empty((n, m), dtype=np.float32)
    for i in range(n):
        xs = shared if iid else rng.standard_normal(d)
        xs = xs / np.linalg.norm(xs)
        prob = 1.0 / (1.0 + np.exp(-(A[i, :, :d].astype(np.float64) @ xs)))
        y[i] = np.where(rng.uniform(size=m) <= prob, 1.0, -1.0)
    return np.ascontiguousarray(A), np.ascontiguousarray(y)
