"""Seeded synthetic inputs drawn directly on a CUDA device (bench-scale workloads).

Same recipe as `workloads.synth` (Haar-orthonormal factors, power-law spectrum,
N(0,1) hidden states and queries rounded to bf16) but generated with torch on the
device, because the full-size configurations hold billions of values.  The
streams differ from the numpy ones; a test that needs the oracle's opinion copies
the drawn inputs back to the host.  No arithmetic of the method lives here.
"""
from __future__ import annotations

import torch

from .synth import BASE_SEED

_TAGS = {"U": 1, "V": 2, "X": 3, "Q": 4, "C": 5}


def _gen(device, *key):
    g = torch.Generator(device=device)
    seed = BASE_SEED
    for k in key:
        seed = (seed * 1000003 + int(k) + 12345) % (2 ** 62)
    g.manual_seed(seed)
    return g


def haar_orthonormal(rows, cols, device, *key):
    """rows x cols fp32 matrix with orthonormal columns (QR of a Gaussian, signs fixed)."""
    g = torch.randn(rows, cols, generator=_gen(device, *key), device=device, dtype=torch.float32)
    q, r = torch.linalg.qr(g)
    sgn = torch.sign(torch.diagonal(r))
    sgn[sgn == 0] = 1.0
    return q * sgn[None, :]


def weight_generators(d_model, n, p, layer, which, device):
    """(U [D,n], sigma [n], V [n,n]) with W = U diag(sigma) V^T, sigma_i = i^-p; fp32 on device."""
    w = {"k": 0, "v": 1}[which]
    u = haar_orthonormal(d_model, n, device, layer, w, _TAGS["U"])
    v = haar_orthonormal(n, n, device, layer, w, _TAGS["V"])
    sigma = torch.arange(1, n + 1, device=device, dtype=torch.float32) ** (-float(p))
    return u, sigma, v


def hidden_states(shape, layer, chunk, device):
    """x ~ N(0,1) in bf16; `shape` ends with d_model."""
    g = _gen(device, layer, chunk, _TAGS["X"])
    return torch.randn(*shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def queries(shape, layer, step, device, scale=1.0):
    """q ~ scale * N(0,1) in bf16; shape [batch, H_q, d_h]."""
    g = _gen(device, layer, step, _TAGS["Q"])
    return (scale * torch.randn(*shape, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)


def latents(shape, p, layer, which, device):
    """Synthetic cache rows for tests that start from a filled cache: coordinate i ~ N(0, i^-2p) in bf16, the
    distribution the rows have when the hidden states are N(0, I) and the spectrum is i^-p; `shape` ends with r."""
    w = {"k": 0, "v": 1}[which]
    g = _gen(device, layer, w, _TAGS["C"])
    r = shape[-1]
    sigma = torch.arange(1, r + 1, device=device, dtype=torch.float32) ** (-float(p))
    return (torch.randn(*shape, generator=g, device=device, dtype=torch.float32) * sigma).to(torch.bfloat16)
