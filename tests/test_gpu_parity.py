"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle.

Tolerances (chosen for the arithmetic, not stated by the paper): max over
(sequence, head) rows of ||gpu - oracle||_2 / ||oracle||_2 <= 1e-2 for the bf16 /
fp32-accumulate path and <= 1e-5 for the fp32 debug path; the cache write within
one bf16 unit in the last place of the exactly rounded latent.
"""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu

TOL_BF16 = 1e-2
TOL_FP32 = 1e-5


def _tol(flags):
    return TOL_FP32 if flags & 1 else TOL_BF16


def _check_append(got_rows, want_rows):
    got = np.asarray(got_rows, dtype=np.float64)
    want = np.asarray(want_rows, dtype=np.float64)
    assert np.all(np.abs(got - want) <= H.bf16_ulp(want) * 1.0 + 1e-30)
    # and almost every entry is the exactly rounded one
    assert np.mean(got == want) > 0.98
    assert O.rel_l2_rows(got, want) <= TOL_BF16


def _check_fp32_path(got, want):
    """fp32 debug path, seen through its bf16 output: each element may deviate by the
    final rounding (half a bf16 ulp) plus TOL_FP32 of the row's rms magnitude."""
    rms = np.sqrt(np.mean(want ** 2, axis=-1, keepdims=True))
    assert np.all(np.abs(got - want) <= 0.5 * H.bf16_ulp(want) + TOL_FP32 * rms)


def _xs(lens, D, layer=0):
    return [synth.hidden_states(int(L), D, layer, chunk=100 + s).astype(np.float64) for s, L in enumerate(lens)]


# --------------------------------------------------------------------------- cfg1
@pytest.mark.parametrize("flags", [1, 0])
@pytest.mark.parametrize("q_scale", [1.0, 64.0])
def test_cfg1_tiny_append_then_decode(flags, q_scale):
    import torch
    c = synth.CONFIGS["cfg1_tiny"]
    prob = H.Problem(c.d_model, c.n_q_heads, c.n_kv_heads, c.d_head, c.ranks[0], c.ranks[0], c.rope_theta,
                     c.sigma_p)
    N = c.context
    sess = H.Session(prob, max_pos=N + 1, batch=1, flags=flags)
    x = synth.hidden_states(N + 1, c.d_model, 0).astype(np.float64)      # 128 prefilled + 1 decoded token
    cache, k, v, sl = H.contiguous_cache(sess, 1, N + 1, [N])
    sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(x[:N]), T=N)         # prefill
    sl += 1
    cache.max_seq_len = N + 1
    sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(x[N:]), T=1)         # the decode step's token
    q = synth.queries(1, c.n_q_heads, c.d_head, 0, 0, q_scale).astype(np.float64)
    out = torch.zeros(1, c.n_q_heads, c.d_head, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    ck, cv = H.oracle_latents(prob, [x])
    _check_append(H.host_f64(k[0]), ck[0])
    _check_append(H.host_f64(v[0]), cv[0])
    want = H.oracle_decode(prob, ck, cv, q)
    # chain parity: GPU latents may differ from the oracle's by one rounding in a few entries
    assert O.rel_l2_rows(H.host_f64(out), want) <= TOL_BF16
    sess.close()


# ------------------------------------------------- kernel parity on oracle-made latents
CASES = [
    # D, H_q, H_kv, d_h, r_k, r_v, lens, style
    (256, 4, 2, 64, 32, 32, [129], 0),
    (512, 8, 2, 128, 96, 72, [1, 37, 300, 700], 0),
    (512, 8, 2, 128, 256, 256, [513, 64, 1000], 0),
    (384, 16, 2, 64, 40, 128, [95, 260], 1),
    (512, 8, 1, 128, 128, 8, [333], 0),
    # style 2: no rotation at attention time (plain kernels with an identity rotation table)
    (256, 4, 2, 64, 32, 32, [129], 2),
    (512, 8, 2, 128, 96, 72, [37, 300], 2),
]


@pytest.mark.parametrize("flags", [1, 0])
@pytest.mark.parametrize("case", CASES)
def test_decode_attn_on_oracle_latents_contiguous(case, flags):
    import torch
    D, H_q, H_kv, d_h, r_k, r_v, lens, style = case
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=500000.0, style=style, layer=3)
    b = len(lens)
    n_max = max(lens) + 5
    sess = H.Session(prob, max_pos=n_max, batch=b, flags=flags)
    ck, cv = H.oracle_latents(prob, _xs(lens, D))
    cache, k, v, sl = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    for q_scale in (1.0, 64.0):
        q = synth.queries(b, H_q, d_h, 3, int(q_scale), q_scale).astype(np.float64)
        out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
        assert sess.L.lorc_sync_status(sess.ctx) == 0
        want = H.oracle_decode(prob, ck, cv, q)
        got = H.host_f64(out)
        if flags & 1:
            _check_fp32_path(got, want)
        assert O.rel_l2_rows(got, want) <= TOL_BF16
    sess.close()


@pytest.mark.parametrize("flags", [1, 0])
def test_decode_attn_paged_and_page_permutation(flags):
    import torch
    D, H_q, H_kv, d_h, r = 512, 8, 2, 128, 96
    lens = [200, 65, 64, 449]
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, theta=500000.0, layer=5)
    b = len(lens)
    sess = H.Session(prob, max_pos=512, batch=b, flags=flags)
    ck, cv = H.oracle_latents(prob, _xs(lens, D, 5))
    q = synth.queries(b, H_q, d_h, 5, 0, 8.0).astype(np.float64)
    want = H.oracle_decode(prob, ck, cv, q)
    outs = []
    for order_seed in (11, 12):
        cache, k, v, sl, ptd, pt = H.paged_cache(sess, b, lens, 64, order_seed, ck, cv)
        out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
        assert sess.L.lorc_sync_status(sess.ctx) == 0
        assert O.rel_l2_rows(H.host_f64(out), want) <= _tol(0)
        outs.append(out.clone())
    # the physical page order does not change a single bit
    assert torch.equal(outs[0], outs[1])
    # and the paged result equals the contiguous one bit for bit
    cache, k, v, sl = H.contiguous_cache(sess, b, 512, lens, ck, cv)
    out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
    assert torch.equal(out, outs[0])
    sess.close()


@pytest.mark.parametrize("flags", [1, 0])
def test_split_count_does_not_change_the_result(flags):
    import torch
    D, H_q, H_kv, d_h, r = 512, 8, 2, 128, 64
    lens = [1500, 70]
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, theta=500000.0, layer=6)
    sess = H.Session(prob, max_pos=1536, batch=2, flags=flags)
    ck, cv = H.oracle_latents(prob, _xs(lens, D, 6))
    cache, k, v, sl = H.contiguous_cache(sess, 2, 1536, lens, ck, cv)
    q = synth.queries(2, H_q, d_h, 6, 0, 16.0).astype(np.float64)
    want = H.oracle_decode(prob, ck, cv, q)
    res = []
    for S in (1, 2, 5, 47):
        out = torch.zeros(2, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, n_splits=S)
        assert sess.L.lorc_sync_status(sess.ctx) == 0
        res.append(H.host_f64(out))
        assert O.rel_l2_rows(res[-1], want) <= _tol(0)
    for r_ in res[1:]:
        # fp32 partials merged in a different order: equal up to the bf16 rounding of the output
        assert np.all(np.abs(r_ - res[0]) <= H.bf16_ulp(res[0]) * 1.0)
    sess.close()


@pytest.mark.parametrize("flags", [1, 0])
def test_ragged_batch_equals_each_sequence_alone(flags):
    import torch
    D, H_q, H_kv, d_h, r = 256, 4, 2, 64, 48
    lens = [17, 190, 64]
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, layer=7)
    sess = H.Session(prob, max_pos=256, batch=3, flags=flags)
    ck, cv = H.oracle_latents(prob, _xs(lens, D, 7))
    q = synth.queries(3, H_q, d_h, 7, 0, 4.0)
    cache, k, v, sl = H.contiguous_cache(sess, 3, 256, lens, ck, cv)
    out = torch.zeros(3, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, n_splits=1)
    for s in range(3):
        c1, k1, v1, sl1 = H.contiguous_cache(sess, 1, 256, [lens[s]], [ck[s]], [cv[s]])
        o1 = torch.zeros(1, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, c1, H.dev_bf16(q[s:s + 1]), o1, n_splits=1)
        assert torch.equal(o1[0], out[s])
    sess.close()


# ------------------------------------------------------------------ append
@pytest.mark.parametrize("flags", [1, 0])
@pytest.mark.parametrize("paged", [False, True])
def test_append_prefill_chunks_and_decode_tokens(flags, paged):
    import torch
    D, H_q, H_kv, d_h, r_k, r_v = 512, 8, 2, 128, 96, 72
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, layer=8)
    b, T1, T2 = 3, 70, 1
    sess = H.Session(prob, max_pos=256, batch=b, flags=flags)
    xs = _xs([T1 + T2 + 1] * b, D, 8)
    lens0 = [T1] * b
    if paged:
        cache, k, v, sl, ptd, pt = H.paged_cache(sess, b, [T1 + T2 + 1] * b, 16, 21)
        sl[:] = T1
    else:
        cache, k, v, sl = H.contiguous_cache(sess, b, 128, lens0)
        cache.max_seq_len = 128
    xd = H.dev_bf16(np.stack([x[:T1] for x in xs]))
    sess.L.lorc_append(sess.ctx, 0, cache, xd, T=T1)
    for step in range(2):
        sl += 1
        xd = H.dev_bf16(np.stack([x[T1 + step:T1 + step + 1] for x in xs]))
        sess.L.lorc_append(sess.ctx, 0, cache, xd, T=1)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    ck, cv = H.oracle_latents(prob, xs)
    for s in range(b):
        n_tok = T1 + 2
        if paged:
            gk = O.gather_rows(H.host_f64(k), pt[s], n_tok, 16)
            gv = O.gather_rows(H.host_f64(v), pt[s], n_tok, 16)
        else:
            gk, gv = H.host_f64(k[s, :n_tok]), H.host_f64(v[s, :n_tok])
        _check_append(gk, ck[s][:n_tok])
        _check_append(gv, cv[s][:n_tok])
    # rows past the sequences stay untouched (zero)
    if not paged:
        assert float(k[:, T1 + 2:].abs().max()) == 0.0
    sess.close()


# --------------------------------------------------------------- full-rank mode
@pytest.mark.parametrize("flags", [1, 0])
@pytest.mark.parametrize("style", [0, 1])
def test_full_mode_matches_uncompressed_attention(flags, style):
    import torch
    D, H_q, H_kv, d_h = 256, 8, 2, 64
    lens = [150, 33]
    prob = H.Problem(D, H_q, H_kv, d_h, 128, 128, theta=10000.0, layer=9, style=style)
    b = 2
    sess = H.Session(prob, max_pos=256, batch=b, flags=flags, mode=1)
    xs = _xs([max(lens)] * b, D, 9)
    cache, k, v, sl = H.contiguous_cache(sess, b, 256, [max(lens)] * b)
    sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(np.stack(xs)), T=max(lens))
    sl[:] = torch.tensor(lens, dtype=torch.int32)
    q = synth.queries(b, H_q, d_h, 9, 0, 8.0).astype(np.float64)
    out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    for s in range(b):
        want = O.decode_attn_full(xs[s][:lens[s]], prob.W_k, prob.W_v, q[s], H_kv, prob.theta, style)
        # the cache rounds rotated keys and values to bf16: bf16-level agreement on both paths
        assert O.rel_l2_rows(H.host_f64(out[s]), want) <= TOL_BF16
        # stored keys are the rotated projections
        Kr = O.rope((xs[s] @ prob.W_k).reshape(-1, H_kv, d_h), np.arange(max(lens))[:, None], prob.theta,
                    style).reshape(-1, prob.n)
        assert np.all(np.abs(H.host_f64(k[s, :max(lens)]) - Kr) <= H.bf16_ulp(Kr) + 1e-6)
    sess.close()


def test_full_mode_equals_latent_mode_at_full_rank():
    import torch
    D, H_q, H_kv, d_h = 256, 4, 2, 64
    n = H_kv * d_h
    N = 100
    prob = H.Problem(D, H_q, H_kv, d_h, n, n, layer=10)
    x = _xs([N], D, 10)
    q = synth.queries(1, H_q, d_h, 10, 0, 8.0).astype(np.float64)
    outs = []
    for mode in (0, 1):
        sess = H.Session(prob, max_pos=128, batch=1, mode=mode)
        cache, k, v, sl = H.contiguous_cache(sess, 1, 128, [N])
        sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(x[0][None]), T=N)
        out = torch.zeros(1, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
        assert sess.L.lorc_sync_status(sess.ctx) == 0
        outs.append(H.host_f64(out))
        sess.close()
    # W (bf16) and A.B (bf16 factors) differ by rounding only
    assert O.rel_l2_rows(outs[0], outs[1]) <= 2 * TOL_BF16
    want = O.decode_attn_full(x[0], prob.W_k, prob.W_v, q[0], H_kv, prob.theta)
    assert O.rel_l2_rows(outs[1][0], want) <= TOL_BF16


# ------------------------------------------------------------ host-buffer entry
def test_decode_step_host_equals_device_calls():
    import torch
    D, H_q, H_kv, d_h, r = 256, 4, 2, 64, 32
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, layer=11)
    b, N = 2, 40
    sess = H.Session(prob, max_pos=64, batch=b)
    xs = _xs([N + 1] * b, D, 11)
    q = synth.queries(b, H_q, d_h, 11, 0, 4.0)
    res = []
    for use_host in (False, True):
        cache, k, v, sl = H.contiguous_cache(sess, b, 64, [N] * b)
        cache.max_seq_len = 64
        sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(np.stack([x[:N] for x in xs])), T=N)
        sl += 1
        xn = np.stack([x[N] for x in xs])
        if use_host:
            xh = torch.from_numpy(xn.astype(np.float32)).to(torch.bfloat16).pin_memory()
            qh = torch.from_numpy(q).to(torch.bfloat16).pin_memory()
            oh = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16).pin_memory()
            sess.L.lorc_decode_step_host(sess.ctx, 0, cache, xh, qh, oh)
            assert sess.L.lorc_sync_status(sess.ctx) == 0
            res.append(oh.clone())
        else:
            sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(xn), T=1)
            out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
            sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out)
            assert sess.L.lorc_sync_status(sess.ctx) == 0
            res.append(out.cpu())
    assert torch.equal(res[0], res[1])
    ck, cv = H.oracle_latents(prob, xs)
    want = H.oracle_decode(prob, ck, cv, q.astype(np.float64))
    assert O.rel_l2_rows(H.host_f64(res[1]), want) <= TOL_BF16
    sess.close()


# -------------------------------------------------------------- error behaviour
def test_errors_are_reported_not_raised_on_the_device():
    import torch
    L = H.lib()
    D, H_q, H_kv, d_h, r = 256, 4, 2, 64, 32
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, layer=12)
    sess = H.Session(prob, max_pos=64, batch=2)
    ck, cv = H.oracle_latents(prob, _xs([10, 10], D, 12))
    q = H.dev_bf16(synth.queries(2, H_q, d_h, 12, 0))
    out = torch.ones(2, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    # an empty sequence: zeros and status EMPTY; the other sequence is still served
    cache, k, v, sl = H.contiguous_cache(sess, 2, 64, [0, 10], ck, cv)
    cache.max_seq_len = 10
    L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
    assert L.lorc_sync_status(sess.ctx) == L.LORC_ERR_EMPTY
    assert float(out[0].abs().max()) == 0.0 and float(out[1].abs().max()) > 0.0
    assert L.lorc_sync_status(sess.ctx) == 0                       # the word was cleared
    # a page index outside the pool is caught by the kernel, not dereferenced
    cache, k, v, sl, ptd, pt = H.paged_cache(sess, 2, [10, 10], 16, 31, ck, cv)
    ptd[1, 0] = 10 ** 6
    L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
    assert L.lorc_sync_status(sess.ctx) == L.LORC_ERR_CAPACITY
    # host-side argument checks
    with pytest.raises(L.LorcError) as e:
        L.lorc_decode_attn(sess.ctx, 3, cache, q, out)
    assert e.value.code == L.LORC_ERR_LAYER
    cache.max_seq_len = 10 ** 6
    with pytest.raises(L.LorcError) as e:
        L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
    assert e.value.code == L.LORC_ERR_ARG
    cache.max_seq_len = 10
    L.lorc_set_workspace(sess.ctx, None)
    with pytest.raises(L.LorcError) as e:
        L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
    assert e.value.code == L.LORC_ERR_WORKSPACE
    with pytest.raises(L.LorcError) as e:
        L.lorc_load_factors(sess.ctx, 0, 0, 12, 32, *sess.dev)     # rank not a multiple of 8
    assert e.value.code == L.LORC_ERR_ARG
    sess.close()


@pytest.mark.parametrize("flags", [1, 0])
def test_latent_output_entry_plain_kernels(flags):
    """lorc_decode_attn_latent_out on the plain kernels (merge without up-projection)."""
    import torch
    D, H_q, H_kv, d_h, r_k, r_v = 256, 4, 2, 64, 40, 24
    lens = [150, 33]
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=10000.0, layer=11)
    sess = H.Session(prob, max_pos=160, batch=2, flags=flags)
    ck, cv = H.oracle_latents(prob, _xs(lens, D, 11))
    held = H.contiguous_cache(sess, 2, 160, lens, ck, cv)
    q = synth.queries(2, H_q, d_h, 11, 0, 8.0).astype(np.float64)
    o_lat = torch.zeros(2, H_q, r_v, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn_latent_out(sess.ctx, 0, held[0], H.dev_bf16(q), o_lat, n_splits=3)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    for s in range(2):
        want = O.decode_attn_latent_out(ck[s], cv[s], prob.B_k, q[s], H_kv, prob.theta)
        assert O.rel_l2_rows(H.host_f64(o_lat[s]), want) <= TOL_BF16
    # an uncompressed layer has no latent output
    full = H.Session(prob, max_pos=160, batch=2, flags=flags, mode=1)
    heldf = H.contiguous_cache(full, 2, 160, lens)
    with pytest.raises(sess.L.LorcError) as e:
        sess.L.lorc_decode_attn_latent_out(full.ctx, 0, heldf[0], H.dev_bf16(q), o_lat)
    assert e.value.code == sess.L.LORC_ERR_UNSUPPORTED
    full.close()
    sess.close()


def test_fp32_debug_path_one_sequence_of_32768_tokens():
    """The plain fp32 kernels over one long sequence (the context length of the long-context configuration) at a
    small rank, element by element: 256 context splits, 2048 tiles, positions up to 32767 in the rotation table."""
    import torch
    N, D, H_q, H_kv, d_h, r_k, r_v = 32768, 256, 8, 2, 64, 32, 24
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=500000.0, layer=9)
    sess = H.Session(prob, max_pos=N, batch=1, flags=H.lib().LORC_FLAG_DEBUG_FP32)
    # latent rows seeded directly (coordinate i of a row ~ N(0, sigma_i^2), what x A gives for x ~ N(0, I)), bf16-exact
    rng = np.random.default_rng(99)
    ck = [synth.to_bf16_exact(rng.standard_normal((N, r_k)) * (np.arange(1, r_k + 1) ** -0.8))]
    cv = [synth.to_bf16_exact(rng.standard_normal((N, r_v)) * (np.arange(1, r_v + 1) ** -0.8))]
    held = H.contiguous_cache(sess, 1, N, [N], ck, cv)
    for q_scale in (1.0, 64.0):
        q = synth.queries(1, H_q, d_h, 9, int(q_scale), q_scale).astype(np.float64)
        out = torch.zeros(1, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, held[0], H.dev_bf16(q), out)
        assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
        assert sess.L.lorc_last_path(sess.ctx) == 1
        want = H.oracle_decode(prob, ck, cv, q)
        _check_fp32_path(H.host_f64(out), want)
    sess.close()
