"""The progressive compression schedule (Sec. 3.2, Eq. "dc", the first loops of Algorithm 1): the oracle's functions
against what the mathematics fixes, and the product's host-side implementation (torch) against the oracle.

Pins of the oracle: the condition number against its definition ||A||_2 ||A^-1||_2 and against the closed form n^p of
the synthetic spectra; the perturbation inequality the section states; the cumulative product against a brute-force
product; Eq. "dc" at its end points, its linearity in log kappa~, and, for equally conditioned layers, against the
closed-form rank list of the benchmark configurations; the skip threshold.
"""
import math

import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth


def _weight(D, n, p, layer, which="k"):
    U, s, V = synth.synth_weight_factors(D, n, p, layer, which)
    return (U * s) @ V.T


def test_condition_number_is_norm_times_inverse_norm():
    rng = np.random.default_rng(5)
    A = rng.standard_normal((7, 7))
    want = np.linalg.norm(A, 2) * np.linalg.norm(np.linalg.inv(A), 2)
    assert abs(O.condition_number(A) - want) <= 1e-10 * want


@pytest.mark.parametrize("n,p", [(64, 0.8), (128, 0.7)])
def test_condition_number_of_power_law_spectrum(n, p):
    # sigma_i = i^-p, i = 1..n  =>  kappa = n^p, whatever the orthonormal factors are
    W = _weight(3 * n, n, p, layer=2)
    assert abs(O.condition_number(W) - n ** p) <= 1e-9 * n ** p


def test_perturbation_bound_of_the_condition_number():
    # ||db|| / ||b|| <= kappa(A) ||dx|| / ||x||  (Sec. 3.2), for b = A x
    rng = np.random.default_rng(6)
    A = rng.standard_normal((9, 9))
    kappa = O.condition_number(A)
    for _ in range(200):
        x, dx = rng.standard_normal(9), 1e-3 * rng.standard_normal(9)
        b, db = A @ x, A @ dx
        assert np.linalg.norm(db) / np.linalg.norm(b) <= kappa * np.linalg.norm(dx) / np.linalg.norm(x) * (1 + 1e-12)


def test_cumulative_condition_is_the_product_from_l_to_the_last_layer():
    kk = np.array([3.0, 1.5, 7.0, 2.0])
    kv = np.array([2.0, 4.0, 1.25, 5.0])
    got = np.exp(O.cumulative_log_condition(kk, kv))
    for l in range(4):
        want = np.prod(kk[l:]) * np.prod(kv[l:])
        assert abs(got[l] - want) <= 1e-12 * want
    assert np.all(np.diff(got) <= 0)          # every kappa >= 1: deeper layers accumulate less


def test_compression_dimension_end_points_and_linearity():
    lk = np.array([9.0, 7.5, 4.0, 3.0, 1.0])
    d = O.compression_dimensions(lk, d_min=256, d_max=1024)
    assert d[0] == 1024 and d[-1] == 256
    # linear in log kappa~: equal steps in lk give equal steps in d
    slope = (1024 - 256) / (9.0 - 1.0)
    assert np.allclose(d, 256 + slope * (lk - 1.0), atol=1e-9)
    # order-preserving: more sensitive layers keep more dimensions
    assert np.all(np.diff(d) <= 0)
    # all layers equally sensitive: nothing to interpolate, d_max everywhere
    assert np.all(O.compression_dimensions(np.full(4, 2.0), 256, 1024) == 1024)


@pytest.mark.parametrize("name,d_min,d_max", [
    ("cfg2_8b_progressive", 0.4 * 1024, 0.9 * 1024),       # retained fractions 0.9 (first layer) ... 0.4 (last)
    ("cfg4_70b_progressive", 0.35 * 1024, 0.85 * 1024),
])
def test_equal_layers_reproduce_the_benchmark_rank_lists(name, d_min, d_max):
    # Every layer of the synthetic models has the same spectrum, so log kappa~_l falls linearly with the layer and
    # Eq. "dc", rounded to multiples of 32, must give the closed-form rank list of the configuration.
    shape = synth.CONFIGS[name]
    L = shape.n_layers
    kappa = np.full(L, float(shape.n) ** shape.sigma_p)
    d, skip = O.progressive_schedule(kappa, kappa, d_min, d_max, quantum=32)
    assert tuple(int(x) for x in d) == tuple(shape.ranks)
    assert not skip.any()


def test_threshold_skips_the_most_sensitive_layers():
    kk = np.array([2.0, 2.0, 2.0, 2.0])
    kv = np.array([3.0, 3.0, 3.0, 3.0])
    lk = O.cumulative_log_condition(kk, kv)          # log 6 * (4, 3, 2, 1)
    d, skip = O.progressive_schedule(kk, kv, 64, 128, quantum=8, log_threshold=2.5 * math.log(6.0))
    assert list(skip) == [True, True, False, False]
    assert list(d) == [128, 104, 88, 64]            # 128 - 64 * (0, 1/3, 2/3, 1), to multiples of 8
    assert np.allclose(lk, math.log(6.0) * np.array([4, 3, 2, 1]))


def test_host_schedule_matches_the_oracle():
    torch = pytest.importorskip("torch")
    from paper_2410_03111_b200 import host
    L, D, n = 5, 96, 48
    ps = [0.9, 0.5, 0.8, 0.6, 0.7]
    Wk = [_weight(D, n, ps[l], l, "k") for l in range(L)]
    Wv = [_weight(D, n, ps[(l + 2) % L], l, "v") for l in range(L)]
    kk = np.array([O.condition_number(w) for w in Wk])
    kv = np.array([O.condition_number(w) for w in Wv])
    got_k = host.condition_numbers([torch.from_numpy(w) for w in Wk]).numpy()
    assert np.allclose(got_k, kk, rtol=1e-9)
    lk = O.cumulative_log_condition(kk, kv)
    got_lk = host.cumulative_log_condition(torch.from_numpy(kk), torch.from_numpy(kv)).numpy()
    assert np.allclose(got_lk, lk, rtol=1e-12)
    assert np.allclose(host.compression_dims(torch.from_numpy(lk), 16, 48).numpy(), O.compression_dimensions(lk, 16, 48))
    thr = float(np.sort(lk)[-2])            # exactly one layer above the threshold
    d, skip = O.progressive_schedule(kk, kv, 16, 48, quantum=8, log_threshold=thr)
    plan = host.make_schedule([torch.from_numpy(w) for w in Wk], [torch.from_numpy(w) for w in Wv], 16, 48, quantum=8,
                              log_threshold=thr)
    assert [m for m, _ in plan] == ["full" if s else "latent" for s in skip]
    assert [r for m, r in plan if m == "latent"] == [int(x) for x, s in zip(d, skip) if not s]
    assert sum(skip) == 1


def test_host_factorize_agrees_with_the_oracle_product():
    # a numerical SVD is unique only up to signs, so compare A B (and the spectrum carried by A), not A or B
    torch = pytest.importorskip("torch")
    from paper_2410_03111_b200 import host
    W = _weight(80, 40, 0.8, 3)
    A, B = host.factorize(torch.from_numpy(W), 24)
    Ao, Bo = O.truncated_svd_factors(W, 24)
    got = A.double().numpy() @ B.double().numpy()
    want = Ao @ Bo
    assert np.max(np.abs(got - want)) <= 2.0 ** -7 * np.max(np.abs(want))      # bf16 factors
