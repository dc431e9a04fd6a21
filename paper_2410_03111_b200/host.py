"""Host-side preprocessing: the compression schedule and the factors the library takes.

One-time set-up work, done with torch on whatever device holds the weights; none of it
is on the decode path.
  - the progressive schedule (Sec. 3.2 and the first two loops of Algorithm 1): condition
    numbers of W_k, W_v, cumulative condition numbers from layer l to the last layer, the
    per-layer compression dimension of Eq. "dc", and the skip threshold;
  - the factors (Sec. 3.1 and Algorithm 1, "Matrix Compression": W ~= U_r Sigma_r V_r^T,
    with Sigma kept on the cached side).
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


# ----------------------------------------------------------------------------- schedule
def singular_values(weights):
    """Singular values of a list of weights [D, n] (or one stacked tensor [L, D, n]), descending, as fp64 [L, min(D, n)].
    Equal shapes are decomposed in one batched call on the tensor's device."""
    W = weights if torch.is_tensor(weights) else torch.stack([w for w in weights])
    return torch.linalg.svdvals(W.double())


def condition_numbers(weights):
    """kappa(W) = sigma_max / sigma_min of every weight (Sec. 3.2), fp64 [L]."""
    s = singular_values(weights)
    return s[:, 0] / s[:, -1]


def cumulative_log_condition(kappa_k, kappa_v):
    """log kappa~_l = sum over j >= l of log kappa(W_k^j) + log kappa(W_v^j)  (Sec. 3.2, cumulative condition number;
    in logs, since the product overflows for deep models and Eq. "dc" only needs logs)."""
    lk = torch.log(kappa_k.double()) + torch.log(kappa_v.double())
    return torch.flip(torch.cumsum(torch.flip(lk, [0]), 0), [0])


def compression_dims(log_kappa_tilde, d_min, d_max):
    """Eq. "dc": d_max for the most sensitive layer, d_min for the least, linear in log kappa~ between (real-valued)."""
    hi, lo = log_kappa_tilde.max(), log_kappa_tilde.min()
    if float(hi) == float(lo):
        return torch.full_like(log_kappa_tilde, float(d_max))
    return d_max * (1.0 - (hi - log_kappa_tilde) / (hi - lo) * (1.0 - float(d_min) / float(d_max)))


def make_schedule(W_k, W_v, d_min, d_max, quantum=32, log_threshold=None):
    """The per-layer plan of Algorithm 1 for the key and value weights W_k, W_v (lists of [D, n] tensors):
    a list of (mode, rank) with mode "latent" (compress to `rank`: Eq. "dc" rounded to the nearest multiple of `quantum`) or
    "full" (cumulative condition number above the threshold, given on the log scale: the layer keeps an ordinary
    cache).  quantum must be a multiple of 8, the granularity lorc_load_factors accepts."""
    if quantum % 8:
        raise ValueError("quantum must be a multiple of 8")
    lk = cumulative_log_condition(condition_numbers(W_k), condition_numbers(W_v))
    d = compression_dims(lk, d_min, d_max)
    d = torch.clamp(torch.round(d / quantum) * quantum, min=quantum).to(torch.int64)      # ties to even
    plan = []
    for l in range(d.shape[0]):
        skip = log_threshold is not None and float(lk[l]) > float(log_threshold)
        plan.append(("full", None) if skip else ("latent", int(d[l])))
    return plan
