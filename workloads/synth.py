"""Seeded synthetic inputs for latent-KV decode attention workloads (host side).

Nothing here belongs to the compression method: the functions draw random
matrices and vectors and list workload shapes.  Weight matrices are described by
their generating factors (U, sigma, V) with W = U diag(sigma) V^T, so that the
singular value decomposition of every synthetic weight is known in closed form.

Every draw is keyed by (base_seed, layer, stream tag, ...) through
numpy's SeedSequence + Philox, so any slice of a workload can be regenerated
independently of the rest.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Tuple

import numpy as np

BASE_SEED = 20241003

# stream tags (kept small and fixed so seeds never collide)
_TAG_U = 1
_TAG_V = 2
_TAG_X = 3
_TAG_Q = 4
_TAG_LEN = 5
_TAG_PAGE = 6
_TAG_MISC = 7


def _rng(*key: int) -> np.random.Generator:
    ss = np.random.SeedSequence([int(k) & 0xFFFFFFFF for k in key])
    return np.random.Generator(np.random.Philox(ss))


def to_bf16_exact(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); return float32.

    Used to make *inputs* that a bf16 device buffer holds exactly.  Works on the
    float32 bit pattern: add 0x7FFF + lsb, then clear the low 16 bits.
    """
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(f.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-exact float32 values (for upload)."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    return (f.view(np.uint32) >> 16).astype(np.uint16).reshape(f.shape)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    """float32 values of bf16 bit patterns."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).reshape(b.shape)


def haar_orthonormal(rows: int, cols: int, *key: int) -> np.ndarray:
    """rows x cols matrix with orthonormal columns, Haar distributed (fp64).

    QR of a Gaussian matrix with the signs of diag(R) folded into Q.
    """
    assert rows >= cols
    g = _rng(*key).standard_normal((rows, cols))
    qm, rm = np.linalg.qr(g)
    sgn = np.sign(np.diag(rm))
    sgn[sgn == 0] = 1.0
    return qm * sgn[None, :]


def spectrum(n: int, p: float) -> np.ndarray:
    """Power-law singular values sigma_i = i^-p, i = 1..n."""
    return np.arange(1, n + 1, dtype=np.float64) ** (-float(p))


def synth_weight_factors(d_model: int, n: int, p: float, layer: int, which: str,
                         base_seed: int = BASE_SEED):
    """Generating factors (U [D,n], sigma [n], V [n,n]) of one synthetic weight.

    which is 'k' or 'v'.  The weight itself is U @ diag(sigma) @ V.T.
    """
    w = {"k": 0, "v": 1}[which]
    u = haar_orthonormal(d_model, n, base_seed, layer, w, _TAG_U)
    v = haar_orthonormal(n, n, base_seed, layer, w, _TAG_V)
    return u, spectrum(n, p), v


def hidden_states(n_tok: int, d_model: int, layer: int, chunk: int = 0,
                  base_seed: int = BASE_SEED) -> np.ndarray:
    """x ~ N(0,1), rounded to bf16; float32 [n_tok, d_model]."""
    g = _rng(base_seed, layer, chunk, _TAG_X)
    return to_bf16_exact(g.standard_normal((n_tok, d_model), dtype=np.float32))


def queries(batch: int, n_q_heads: int, d_head: int, layer: int, step: int,
            scale: float = 1.0, base_seed: int = BASE_SEED) -> np.ndarray:
    """q ~ scale * N(0,1), rounded to bf16; float32 [batch, H_q, d_h]."""
    g = _rng(base_seed, layer, step, _TAG_Q)
    return to_bf16_exact(scale * g.standard_normal((batch, n_q_heads, d_head), dtype=np.float32))


def ragged_lengths(batch: int, lo: int, hi: int, base_seed: int = BASE_SEED) -> np.ndarray:
    """Context lengths uniform on {lo..hi}; int32 [batch]."""
    return _rng(base_seed, _TAG_LEN).integers(lo, hi + 1, size=batch).astype(np.int32)


def page_order(n_pages: int, base_seed: int = BASE_SEED) -> np.ndarray:
    """A seeded random permutation of physical page indices; int32 [n_pages]."""
    return _rng(base_seed, _TAG_PAGE).permutation(n_pages).astype(np.int32)


def gaussian(shape, *key: int) -> np.ndarray:
    """Plain fp64 standard normal draws for small tests."""
    return _rng(BASE_SEED, _TAG_MISC, *key).standard_normal(shape)


def rank_schedule(n_layers: int, n: int, c0: float, slope: float = 0.5, q: int = 32):
    """Per-layer ranks r_l = q*round(n*(c0 - slope*l/(L-1))/q), l = 0..L-1."""
    out = []
    for l in range(n_layers):
        frac = c0 - slope * l / (n_layers - 1) if n_layers > 1 else c0
        out.append(int(q * round(n * frac / q)))
    return tuple(out)


@dataclass(frozen=True)
class Shape:
    """One workload: model dimensions, ranks per layer, batch and context."""
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    rope_theta: float
    sigma_p: float
    ranks: Tuple[int, ...]
    batch: int
    context: int            # tokens prefilled per sequence (max for ragged)
    decode_steps: int
    paged: bool = False
    page_size: int = 64
    ragged: Tuple[int, int] = field(default=(0, 0))   # (lo, hi) when lengths are drawn

    @property
    def n(self) -> int:
        return self.n_kv_heads * self.d_head

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


def _configs():
    c = {}
    c["cfg1_tiny"] = Shape("cfg1_tiny", 1, 256, 4, 2, 64, 10000.0, 0.8, (32,), 1, 128, 1)
    c["cfg2_8b_progressive"] = Shape(
        "cfg2_8b_progressive", 32, 4096, 32, 8, 128, 500000.0, 0.8,
        rank_schedule(32, 1024, 0.9), 16, 4096, 64)
    c["cfg3_8b_long"] = Shape(
        "cfg3_8b_long", 32, 4096, 32, 8, 128, 500000.0, 0.8, (256,) * 32, 4, 32768, 32)
    c["cfg4_70b_progressive"] = Shape(
        "cfg4_70b_progressive", 80, 8192, 64, 8, 128, 500000.0, 0.7,
        rank_schedule(80, 1024, 0.85), 8, 8192, 32)
    for r in (128, 256, 384, 1024):
        c[f"cfg5_ragged_r{r}"] = Shape(
            f"cfg5_ragged_r{r}", 32, 4096, 32, 8, 128, 500000.0, 0.8, (r,) * 32, 64, 16384, 1,
            paged=True, page_size=64, ragged=(512, 16384))
    return c


CONFIGS = _configs()
