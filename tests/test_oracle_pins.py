"""Pins for the CPU oracle: each function is checked against something the paper
or the mathematics fixes, not against itself."""
import cmath
import math
import os

import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ rounding
def test_bf16_round_known_values():
    # spacing in [1,2) is 2^-7; exact ties go to the even significand
    x = np.array([1.0, 1 + 2 ** -8, 1 + 3 * 2 ** -8, 1 + 2 ** -8 + 2 ** -20, -(1 + 2 ** -8),
                  0.0, 2 ** -126, 2 ** -133, 2 ** -134, 0.75 * 2 ** -133, 3.0e38, 3.39e38, 3.4e38])
    want = np.array([1.0, 1.0, 1 + 2 ** -6, 1 + 2 ** -7, -1.0,
                     0.0, 2 ** -126, 2 ** -133, 0.0, 2 ** -133,
                     float(np.ldexp(226.0, 120)), float(np.ldexp(255.0, 120)), np.inf])
    got = O.bf16_round(x)
    assert np.array_equal(got, want)


def test_bf16_round_matches_library_cast():
    torch = pytest.importorskip("torch")
    x = synth.gaussian((20000,), 11).astype(np.float32) * np.float32(37.0)
    lib = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.bf16_round(x.astype(np.float64)), lib)
    # and the input generator's rounding agrees with both
    assert np.array_equal(synth.to_bf16_exact(x).astype(np.float64), lib)


# ------------------------------------------------------------- factorisation
def _tail(n, p, r):
    i = np.arange(r + 1, n + 1, dtype=np.float64)
    return float(np.sum(i ** (-2.0 * p)))


def _total(n, p):
    return _tail(n, p, 0)


@pytest.mark.parametrize("D,n,p,r,tail,eps", [
    (256, 128, 0.8, 32, 0.1159262, 0.2297970),
    (320, 128, 0.7, 96, None, None),
])
def test_eckart_young_closed_form(D, n, p, r, tail, eps):
    U, s, V = synth.synth_weight_factors(D, n, p, layer=0, which="k")
    W = (U * s) @ V.T
    t = _tail(n, p, r)
    if tail is not None:
        assert abs(t - tail) < 5e-8          # closed-form value for sigma_i = i^-0.8
    for A, B in (O.truncated_svd_factors(W, r), O.factors_from_generators(U, s, V, r)):
        assert A.shape == (D, r) and B.shape == (r, n)
        err2 = float(np.sum((W - A @ B) ** 2))
        assert abs(err2 - t) < 1e-10
        e = O.relative_frobenius_error(W, A @ B)
        assert abs(e - math.sqrt(t / _total(n, p))) < 1e-10
        if eps is not None:
            assert abs(e - eps) < 5e-8
        # Sigma sits on the cached factor A; B has orthonormal rows
        assert np.allclose(B @ B.T, np.eye(r), atol=1e-10)
        assert np.allclose(np.sqrt(np.sum(A * A, axis=0)), s[:r], atol=1e-10)


def test_svd_recovers_generating_spectrum():
    U, s, V = synth.synth_weight_factors(192, 64, 0.8, layer=3, which="v")
    W = (U * s) @ V.T
    sv = np.linalg.svd(W, compute_uv=False)
    assert np.allclose(sv, s, rtol=0, atol=1e-12)
    A, B = O.truncated_svd_factors(W, 64)
    assert np.allclose(A @ B, W, atol=1e-12)          # full rank is exact
    A1, B1 = O.truncated_svd_factors(W, 24)
    A2, B2 = O.factors_from_generators(U, s, V, 24)
    assert np.allclose(A1 @ B1, A2 @ B2, atol=1e-12)  # unique product, factors up to sign


def test_frobenius_error_definition():
    M = np.array([[3.0, 0.0], [0.0, 4.0]])
    Mh = np.array([[3.0, 0.0], [0.0, 0.0]])
    assert O.relative_frobenius_error(M, Mh) == pytest.approx(4.0 / 5.0, abs=1e-15)


def test_theorem1_bound_and_tightness():
    D, n, p, r = 160, 96, 0.8, 40
    U, s, V = synth.synth_weight_factors(D, n, p, layer=1, which="k")
    W = (U * s) @ V.T
    A, B = O.factors_from_generators(U, s, V, r)
    x = synth.gaussian((64, D), 5)
    err = np.linalg.norm(x @ W - O.append_latent(x, A) @ B, axis=1)
    assert np.all(err <= s[r] * np.linalg.norm(x, axis=1) * (1 + 1e-12))
    # equality along the first dropped left singular vector
    x1 = U[:, r][None, :]
    e1 = np.linalg.norm(x1 @ W - O.append_latent(x1, A) @ B)
    assert e1 == pytest.approx(s[r], rel=1e-10)
    # and no error along a kept direction
    x0 = U[:, 0][None, :]
    assert np.linalg.norm(x0 @ W - O.append_latent(x0, A) @ B) < 1e-12


def test_latent_coordinates_have_variance_sigma_squared():
    # x ~ N(0, I) and orthonormal U  =>  (x U)_i ~ N(0,1) independent, latent_i ~ N(0, sigma_i^2)
    D, n, p, r = 128, 64, 0.8, 16
    U, s, V = synth.synth_weight_factors(D, n, p, layer=2, which="k")
    A, _ = O.factors_from_generators(U, s, V, r)
    x = synth.gaussian((40000, D), 9)
    c = O.append_latent(x, A)
    var = np.var(c, axis=0)
    assert np.allclose(var, s[:r] ** 2, rtol=0.05)
    cc = np.corrcoef(c.T)
    assert np.max(np.abs(cc - np.eye(r))) < 0.03


def test_append_is_plain_matmul_and_bf16_rounded():
    x = np.array([[1.0, 2.0, -1.0]])
    A = np.array([[1.0, 0.5], [0.25, 1.0], [1.0, 2 ** -9]])
    c = O.append_latent(x, A)
    assert np.array_equal(c, np.array([[0.5, 2.5 - 2 ** -9]]))
    assert np.array_equal(O.append_latent_bf16(x, A), np.array([[0.5, 2.5]]))


# ---------------------------------------------------------------------- RoPE
@pytest.mark.parametrize("style", [O.ROPE_HALF_SPLIT, O.ROPE_INTERLEAVED])
def test_rope_complex_closed_form(style):
    d, theta = 16, 10000.0
    v = synth.gaussian((5, d), 21)
    pos = np.array([0, 1, 7, 1000, 32767])
    got = O.rope(v, pos, theta, style)
    for t in range(5):
        for j in range(d // 2):
            ia, ib = (j, j + d // 2) if style == O.ROPE_HALF_SPLIT else (2 * j, 2 * j + 1)
            z = complex(v[t, ia], v[t, ib]) * cmath.exp(1j * pos[t] * theta ** (-2.0 * j / d))
            assert got[t, ia] == pytest.approx(z.real, abs=1e-9)
            assert got[t, ib] == pytest.approx(z.imag, abs=1e-9)
    assert np.array_equal(got[0], v[0])                           # R(0) = I
    assert np.allclose(np.linalg.norm(got, axis=1), np.linalg.norm(v, axis=1))


def test_rope_unit_vector_first_pair():
    # j = 0 has frequency 1: e_0 at position p goes to (cos p) e_0 + (sin p) e_{d/2}
    d = 8
    e0 = np.zeros(d)
    e0[0] = 1.0
    out = O.rope(e0[None, :], np.array([2.0]), 500000.0)[0]
    want = np.zeros(d)
    want[0], want[d // 2] = math.cos(2.0), math.sin(2.0)
    assert np.allclose(out, want, atol=1e-15)
    # the last pair turns by p * theta^(-(d-2)/d)
    e3 = np.zeros(d)
    e3[3] = 1.0
    out = O.rope(e3[None, :], np.array([5.0]), 16.0)[0]
    a = 5.0 * 16.0 ** (-6.0 / 8.0)
    want = np.zeros(d)
    want[3], want[7] = math.cos(a), math.sin(a)
    assert np.allclose(out, want, atol=1e-15)


def test_rope_scores_depend_on_relative_position_only():
    # q_m^T k_n = x^T W_q R_{n-m} W_k^T x_n  (Appendix "Adjusted Position Embedding")
    d, theta = 32, 500000.0
    q = synth.gaussian((d,), 31)
    k = synth.gaussian((d,), 32)
    base = float(O.rope(q[None], np.array([10]), theta)[0] @ O.rope(k[None], np.array([3]), theta)[0])
    for shift in (1, 100, 20000):
        s = float(O.rope(q[None], np.array([10 + shift]), theta)[0]
                  @ O.rope(k[None], np.array([3 + shift]), theta)[0])
        assert s == pytest.approx(base, abs=1e-9)
    rel = float(q @ O.rope(k[None], np.array([3 - 10]), theta)[0])
    assert rel == pytest.approx(base, abs=1e-10)


# ----------------------------------------------------------------- attention
def _brute_force(q_hat, K_hat, V):
    """Textbook softmax(q K^T / sqrt(d)) V with python loops and math.exp."""
    H_q, d = q_hat.shape
    N, H_kv, _ = K_hat.shape
    G = H_q // H_kv
    out = [[0.0] * d for _ in range(H_q)]
    for h in range(H_q):
        g = h // G
        logits = []
        for n in range(N):
            acc = 0.0
            for j in range(d):
                acc += q_hat[h, j] * K_hat[n, g, j]
            logits.append(acc / math.sqrt(d))
        z = sum(math.exp(l) for l in logits)
        for n in range(N):
            w = math.exp(logits[n]) / z
            for j in range(d):
                out[h][j] += w * V[n, g, j]
    return np.array(out)


def test_attention_against_brute_force_and_library():
    torch = pytest.importorskip("torch")
    H_q, H_kv, d, N = 6, 2, 8, 13
    q = synth.gaussian((H_q, d), 41) * 2.0
    K = synth.gaussian((N, H_kv, d), 42)
    V = synth.gaussian((N, H_kv, d), 43)
    got = O.attention_one_query(q, K, V)
    assert np.allclose(got, _brute_force(q, K, V), atol=1e-12)
    # library routine: repeat KV heads per group, fp64 SDPA
    G = H_q // H_kv
    tq = torch.from_numpy(q)[None, :, None, :]                               # [1,H_q,1,d]
    tk = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, 0)[None]  # [1,H_q,N,d]
    tv = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    lib = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, :, 0, :].numpy()
    assert np.allclose(got, lib, atol=1e-12)


def _tiny_problem(D=48, H_q=4, H_kv=2, d=8, N=11, p=0.8, seed=50):
    n = H_kv * d
    Uk, sk, Vk = synth.synth_weight_factors(D, n, p, layer=seed, which="k")
    Uv, sv, Vv = synth.synth_weight_factors(D, n, p, layer=seed, which="v")
    x = synth.gaussian((N, D), seed, 1)
    q = synth.gaussian((H_q, d), seed, 2) * 3.0
    return dict(D=D, H_q=H_q, H_kv=H_kv, d=d, N=N, n=n, Uk=Uk, sk=sk, Vk=Vk, Uv=Uv, sv=sv, Vv=Vv,
                Wk=(Uk * sk) @ Vk.T, Wv=(Uv * sv) @ Vv.T, x=x, q=q)


@pytest.mark.parametrize("style", [O.ROPE_HALF_SPLIT, O.ROPE_INTERLEAVED])
def test_full_rank_equals_uncompressed_attention(style):
    P = _tiny_problem()
    theta = 10000.0
    Ak, Bk = O.factors_from_generators(P["Uk"], P["sk"], P["Vk"], P["n"])
    Av, Bv = O.factors_from_generators(P["Uv"], P["sv"], P["Vv"], P["n"])
    lat = O.decode_attn_latent(O.append_latent(P["x"], Ak), O.append_latent(P["x"], Av), Bk, Bv,
                               P["q"], P["H_kv"], theta, style)
    full = O.decode_attn_full(P["x"], P["Wk"], P["Wv"], P["q"], P["H_kv"], theta, style)
    assert np.max(np.abs(lat - full)) < 1e-12
    # numerical-SVD factors give the same output (factor signs cancel)
    Ak2, Bk2 = O.truncated_svd_factors(P["Wk"], P["n"])
    Av2, Bv2 = O.truncated_svd_factors(P["Wv"], P["n"])
    lat2 = O.decode_attn_latent(O.append_latent(P["x"], Ak2), O.append_latent(P["x"], Av2), Bk2, Bv2,
                                P["q"], P["H_kv"], theta, style)
    assert np.max(np.abs(lat2 - full)) < 1e-11


def test_uncompressed_attention_against_brute_force_with_rope():
    # independent route: rotate with complex arithmetic, attend with python loops
    P = _tiny_problem(N=7)
    theta, d, H_kv = 10000.0, P["d"], P["H_kv"]
    K = (P["x"] @ P["Wk"]).reshape(P["N"], H_kv, d)
    V = (P["x"] @ P["Wv"]).reshape(P["N"], H_kv, d)

    def rot(v, pos):
        out = np.empty_like(v)
        for j in range(d // 2):
            z = complex(v[j], v[j + d // 2]) * cmath.exp(1j * pos * theta ** (-2.0 * j / d))
            out[j], out[j + d // 2] = z.real, z.imag
        return out

    Kr = np.array([[rot(K[t, g], t) for g in range(H_kv)] for t in range(P["N"])])
    qr = np.array([rot(P["q"][h], P["N"] - 1) for h in range(P["H_q"])])
    want = _brute_force(qr, Kr, V)
    got = O.decode_attn_full(P["x"], P["Wk"], P["Wv"], P["q"], H_kv, theta)
    assert np.allclose(got, want, atol=1e-12)
    # identity factors (A = W, B = I) make the latent routine the textbook one
    got2 = O.decode_attn_latent(P["x"] @ P["Wk"], P["x"] @ P["Wv"], np.eye(P["n"]), np.eye(P["n"]),
                                P["q"], H_kv, theta)
    assert np.allclose(got2, want, atol=1e-12)
    # cache-of-rotated-keys pipeline gives the same numbers
    got3 = O.decode_attn_cached_kv(Kr, V, P["q"], theta)
    assert np.allclose(got3, want, atol=1e-12)


def test_special_cases_single_token_zero_query_linearity_groups():
    P = _tiny_problem(N=9)
    r, theta = 6, 10000.0
    Ak, Bk = O.factors_from_generators(P["Uk"], P["sk"], P["Vk"], r)
    Av, Bv = O.factors_from_generators(P["Uv"], P["sv"], P["Vv"], r)
    ck, cv = O.append_latent(P["x"], Ak), O.append_latent(P["x"], Av)
    d, H_kv, G = P["d"], P["H_kv"], P["H_q"] // P["H_kv"]
    # one cached token: softmax weight 1, output = reconstructed value of that token
    o1 = O.decode_attn_latent(ck[:1], cv[:1], Bk, Bv, P["q"], H_kv, theta)
    v0 = (cv[0] @ Bv).reshape(H_kv, d)
    for h in range(P["H_q"]):
        assert np.allclose(o1[h], v0[h // G], atol=1e-13)
    # zero query: uniform weights, output = mean of reconstructed values
    o0 = O.decode_attn_latent(ck, cv, Bk, Bv, np.zeros_like(P["q"]), H_kv, theta)
    vm = (cv @ Bv).reshape(P["N"], H_kv, d).mean(axis=0)
    for h in range(P["H_q"]):
        assert np.allclose(o0[h], vm[h // G], atol=1e-13)
    # linear in C_V
    cv2 = synth.gaussian(cv.shape, 77)
    oa = O.decode_attn_latent(ck, cv, Bk, Bv, P["q"], H_kv, theta)
    ob = O.decode_attn_latent(ck, cv2, Bk, Bv, P["q"], H_kv, theta)
    oc = O.decode_attn_latent(ck, 2.0 * cv - 3.0 * cv2, Bk, Bv, P["q"], H_kv, theta)
    assert np.allclose(oc, 2.0 * oa - 3.0 * ob, atol=1e-12)
    # identical queries inside a GQA group give identical outputs; different groups differ
    q = P["q"].copy()
    q[1] = q[0]
    q[3] = q[2] = q[0]
    og = O.decode_attn_latent(ck, cv, Bk, Bv, q, H_kv, theta)
    assert np.array_equal(og[0], og[1]) and np.array_equal(og[2], og[3])
    assert np.max(np.abs(og[0] - og[2])) > 1e-3


def test_position_shift_invariance_of_output():
    P = _tiny_problem(N=10)
    r, theta = 8, 500000.0
    Ak, Bk = O.factors_from_generators(P["Uk"], P["sk"], P["Vk"], r)
    Av, Bv = O.factors_from_generators(P["Uv"], P["sv"], P["Vv"], r)
    ck, cv = O.append_latent(P["x"], Ak), O.append_latent(P["x"], Av)
    base = O.decode_attn_latent(ck, cv, Bk, Bv, P["q"], P["H_kv"], theta)
    sh = O.decode_attn_latent(ck, cv, Bk, Bv, P["q"], P["H_kv"], theta,
                              positions=np.arange(10) + 12345, q_position=9 + 12345)
    assert np.allclose(base, sh, atol=1e-9)
    # a wrong query position does change the result
    bad = O.decode_attn_latent(ck, cv, Bk, Bv, P["q"], P["H_kv"], theta, q_position=3)
    assert np.max(np.abs(bad - base)) > 1e-4


def test_without_rope_reconstructed_score_equals_absorbed_score():
    # Sec. 3.1: the orthonormal factor can be folded into the query side, s = (B_K,g q_h) . c_n
    P = _tiny_problem(N=12)
    r = 5
    Ak, Bk = O.factors_from_generators(P["Uk"], P["sk"], P["Vk"], r)
    Av, Bv = O.factors_from_generators(P["Uv"], P["sv"], P["Vv"], r)
    ck, cv = O.append_latent(P["x"], Ak), O.append_latent(P["x"], Av)
    d, H_kv, H_q = P["d"], P["H_kv"], P["H_q"]
    G = H_q // H_kv
    got = O.decode_attn_latent(ck, cv, Bk, Bv, P["q"], H_kv, 10000.0, use_rope=False)
    want = np.empty_like(got)
    for h in range(H_q):
        g = h // G
        q_abs = Bk[:, g * d:(g + 1) * d] @ P["q"][h]            # [r]
        s = ck @ q_abs / math.sqrt(d)
        w = np.exp(s - s.max())
        w /= w.sum()
        o_lat = w @ cv                                           # [r_v], value side absorbed too
        want[h] = o_lat @ Bv[:, g * d:(g + 1) * d]
    assert np.allclose(got, want, atol=1e-12)


def test_truncation_changes_logits_by_at_most_theorem1():
    # |s~_n - s_n| <= ||q|| sigma_{r+1} ||x_n|| / sqrt(d): rotations are orthogonal
    P = _tiny_problem(N=16)
    r, theta, d = 4, 10000.0, P["d"]
    Ak, Bk = O.factors_from_generators(P["Uk"], P["sk"], P["Vk"], r)
    ck = O.append_latent(P["x"], Ak)
    pos = np.arange(P["N"])
    K = O.rope((P["x"] @ P["Wk"]).reshape(P["N"], P["H_kv"], d), pos[:, None], theta)
    Kt = O.rope((ck @ Bk).reshape(P["N"], P["H_kv"], d), pos[:, None], theta)
    qh = O.rope(P["q"], np.full((P["H_q"],), P["N"] - 1), theta)
    G = P["H_q"] // P["H_kv"]
    for h in range(P["H_q"]):
        ds = np.abs((K[:, h // G] - Kt[:, h // G]) @ qh[h]) / math.sqrt(d)
        bound = np.linalg.norm(P["q"][h]) * P["sk"][r] * np.linalg.norm(P["x"], axis=1) / math.sqrt(d)
        assert np.all(ds <= bound * (1 + 1e-12))
    assert np.max(np.abs(K - Kt)) > 1e-3          # the truncation is not a no-op


def test_batch_driver_paged_equals_contiguous():
    H_q, H_kv, d, r, b, ps = 4, 2, 8, 6, 3, 4
    n = H_kv * d
    lens = np.array([5, 9, 1])
    Bk = synth.gaussian((r, n), 61)
    Bv = synth.gaussian((r, n), 62)
    ck = synth.gaussian((b, 12, r), 63)
    cv = synth.gaussian((b, 12, r), 64)
    q = synth.gaussian((b, H_q, d), 65)
    ref = O.decode_attn_latent_batch(ck, cv, lens, Bk, Bv, q, H_kv, 10000.0)
    # scatter into a shuffled page pool
    order = synth.page_order(9)
    pt = order.reshape(3, 3)
    pool_k = np.full((9, ps, r), np.nan)
    pool_v = np.full((9, ps, r), np.nan)
    for s in range(b):
        for pg in range(3):
            pool_k[pt[s, pg]] = ck[s, pg * ps:(pg + 1) * ps]
            pool_v[pt[s, pg]] = cv[s, pg * ps:(pg + 1) * ps]
    got = O.decode_attn_latent_batch(pool_k, pool_v, lens, Bk, Bv, q, H_kv, 10000.0,
                                     page_table=pt, page_size=ps)
    assert np.array_equal(got, ref)
    for s in range(b):
        one = O.decode_attn_latent(ck[s, :lens[s]], cv[s, :lens[s]], Bk, Bv, q[s], H_kv, 10000.0)
        assert np.array_equal(one, ref[s])


# -------------------------------------------------------------- memory model
def test_cache_size_model_reproduces_memory_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "memory_table.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for model, b, N, h, d, L, full, ours, ratio, dim, dim_c in rows:
        b, N, h, d, L = int(b), int(N), int(h), int(d), int(L)
        assert h * d == int(dim)
        gib = O.kv_cache_elements(b, N, h, d) * L * 2 / 2 ** 30
        assert gib == pytest.approx(float(full), abs=1e-9)
        assert float(ours) == pytest.approx(float(full) * float(ratio) / 100.0, rel=1e-9)
        # the most compressed layer keeps dim_c of dim columns
        assert O.compression_ratio(int(dim_c), h, d) == pytest.approx(int(dim_c) / int(dim))
        assert O.compression_ratio(int(dim_c), h, d) <= float(ratio) / 100.0


def test_rel_l2_rows_metric():
    want = np.array([[3.0, 4.0], [0.0, 2.0]])
    got = np.array([[3.0, 4.5], [0.0, 2.0]])
    assert O.rel_l2_rows(got, want) == pytest.approx(0.1)


def _golden_eckart_young():
    import os
    rows = []
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "eckart_young.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                n, p, r, t, e = line.split()
                rows.append((int(n), float(p), int(r), float(t), float(e)))
    return rows


# closed-form values for the benchmark spectra (n = 1024: ranks of the 8B and 70B schedules), as listed with the
# workload definitions; the golden file is written by tests/golden/make_eckart_young.py
LISTED = {(128, 0.8, 32): (0.1159262, 0.2297970), (1024, 0.8, 128): (0.0644362, 0.1688638),
          (1024, 0.8, 256): (0.0337240, 0.1221633), (1024, 0.8, 384): (0.0208377, 0.0960276),
          (1024, 0.8, 416): (0.0186425, 0.0908288), (1024, 0.8, 512): (0.0134146, 0.0770479),
          (1024, 0.8, 928): (0.00158316, 0.0264688), (1024, 0.7, 352): (0.0831541, 0.1679115),
          (1024, 0.7, 864): (0.0109796, 0.0610144)}


@pytest.mark.parametrize("n,p,r,tail,eps", _golden_eckart_young())
def test_eckart_young_benchmark_spectra(n, p, r, tail, eps):
    """relative_frobenius_error and factors_from_generators on the benchmark's spectra against the closed form."""
    assert abs(tail - _tail(n, p, r)) <= 1e-12 and abs(eps - math.sqrt(_tail(n, p, r) / _total(n, p))) <= 1e-12
    lt, le = LISTED[(n, p, r)]
    assert abs(tail - lt) <= 5e-8 and abs(eps - le) <= 5e-8
    # square weight (D = n): the error depends on the spectrum alone, so a small D keeps the test fast
    U, s, V = synth.synth_weight_factors(n, n, p, layer=1, which="k")
    W = (U * s) @ V.T
    A, B = O.factors_from_generators(U, s, V, r)
    assert abs(O.relative_frobenius_error(W, A @ B) - eps) <= 1e-9
    assert abs(float(np.sum((W - A @ B) ** 2)) - tail) <= 1e-9


def test_latent_output_times_value_factor_is_the_attention_output():
    """decode_attn_latent_out (Sec. 3.1, the W_o' fold): multiplying by B_V[:, g(h)] gives decode_attn_latent; with a
    single cached token it is that token's latent; its rows are convex combinations of the cached latents."""
    D, H_q, H_kv, d_h, r_k, r_v, N = 96, 8, 2, 16, 24, 20, 37
    n = H_kv * d_h
    Uk, sk, Vk = synth.synth_weight_factors(D, n, 0.8, 4, "k")
    Uv, sv, Vv = synth.synth_weight_factors(D, n, 0.8, 4, "v")
    Ak, Bk = O.factors_from_generators(Uk, sk, Vk, r_k)
    Av, Bv = O.factors_from_generators(Uv, sv, Vv, r_v)
    x = synth.hidden_states(N, D, 4).astype(np.float64)
    q = synth.queries(1, H_q, d_h, 4, 0, 8.0)[0].astype(np.float64)
    ck, cv = O.append_latent(x, Ak), O.append_latent(x, Av)
    for use_rope in (True, False):
        o_lat = O.decode_attn_latent_out(ck, cv, Bk, q, H_kv, 10000.0, use_rope=use_rope)
        full = O.decode_attn_latent(ck, cv, Bk, Bv, q, H_kv, 10000.0, use_rope=use_rope)
        G = H_q // H_kv
        for h in range(H_q):
            g = h // G
            assert np.allclose(o_lat[h] @ Bv[:, g * d_h:(g + 1) * d_h], full[h], atol=1e-12)
        assert np.all(o_lat.min(axis=0) >= cv.min(axis=0) - 1e-12) and np.all(o_lat.max(axis=0) <= cv.max(axis=0) + 1e-12)
    one = O.decode_attn_latent_out(ck[:1], cv[:1], Bk, q, H_kv, 10000.0)
    assert np.allclose(one, np.tile(cv[0], (H_q, 1)), atol=1e-14)


def test_prefill_attention_is_masked_dense_attention():
    """prefill_attn_latent against brute force: reconstruct every key and value, rotate, one dense masked softmax per
    head (query t sees positions <= N - T + t), and against the full-rank uncompressed attention of each prefix."""
    D, H_q, H_kv, d_h, N, T = 48, 4, 2, 8, 11, 5
    n = H_kv * d_h
    Uk, sk, Vk = synth.synth_weight_factors(D, n, 0.8, 6, "k")
    Uv, sv, Vv = synth.synth_weight_factors(D, n, 0.8, 6, "v")
    x = synth.hidden_states(N, D, 6).astype(np.float64)
    q = synth.queries(T, H_q, d_h, 6, 0, 4.0).astype(np.float64)
    for r in (n, 6):
        Ak, Bk = O.factors_from_generators(Uk, sk, Vk, r)
        Av, Bv = O.factors_from_generators(Uv, sv, Vv, r)
        ck, cv = O.append_latent(x, Ak), O.append_latent(x, Av)
        got = O.prefill_attn_latent(ck, cv, Bk, Bv, q, H_kv, 10000.0)
        K = O.rope((ck @ Bk).reshape(N, H_kv, d_h), np.arange(N)[:, None], 10000.0)
        V = (cv @ Bv).reshape(N, H_kv, d_h)
        G = H_q // H_kv
        for t in range(T):
            pos = N - T + t
            qh = O.rope(q[t], np.full((H_q,), pos), 10000.0)
            for h in range(H_q):
                s = K[:, h // G, :] @ qh[h] / math.sqrt(d_h)
                s[pos + 1:] = -np.inf                        # causal mask inside the new chunk
                p = np.exp(s - s.max())
                want = (p / p.sum()) @ V[:, h // G, :]
                assert np.allclose(got[t, h], want, atol=1e-12)
            if r == n:
                # full rank: the uncompressed model's attention for the prefix that ends at this token
                W_k, W_v = (Uk * sk) @ Vk.T, (Uv * sv) @ Vv.T
                assert np.allclose(got[t], O.decode_attn_full(x[:pos + 1], W_k, W_v, q[t], H_kv, 10000.0), atol=1e-10)
        # the last query is the decode query
        assert np.allclose(got[-1], O.decode_attn_latent(ck, cv, Bk, Bv, q[-1], H_kv, 10000.0), atol=1e-14)
