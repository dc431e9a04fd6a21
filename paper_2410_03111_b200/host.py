"""Host-side preprocessing: turning a weight's SVD into the factors the library takes.

One-time set-up work (Sec. 3.1 and Algorithm 1 of the paper: W ~= U_r Sigma_r V_r^T,
with Sigma kept on the cached side), done with torch on whatever device holds the
weights; none of it is on the decode path.
"""
from __future__ import annotations

import torch


def factors_from_svd(U, sigma, V, r):
    """A = U[:, :r] diag(sigma[:r]) [D, r] and B = V[:, :r]^T [r, n], in bf16."""
    A = (U[:, :r] * sigma[None, :r]).to(torch.bfloat16).contiguous()
    B = V[:, :r].t().to(torch.bfloat16).contiguous()
    return A, B


def factorize(W, r):
    """Truncated SVD of W [D, n] (fp32/fp64 tensor) into bf16 factors (A [D, r], B [r, n])."""
    U, s, Vh = torch.linalg.svd(W.double(), full_matrices=False)
    return factors_from_svd(U, s, Vh.t(), r)


def dense_weight(U, sigma, V):
    """W = U diag(sigma) V^T in bf16 (for layers kept uncompressed)."""
    return ((U * sigma[None, :]) @ V.t()).to(torch.bfloat16).contiguous()
