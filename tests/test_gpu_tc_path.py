"""GPU parity of the tensor-core (tcgen05) decode path against the fp64 oracle, through the C ABI.

Shapes here have the 8B head geometry (32 query heads, 8 KV heads of 128) so that the library picks
its tensor-core kernels; each test asserts that it did.  Tolerance: max relative L2 error per
(sequence, head) row <= 1e-2 (bf16 operands, fp32 accumulation).
"""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu
TOL = 1e-2
GEOM = dict(D=1024, H_q=32, H_kv=8, d_h=128)
_PROBS = {}


def _prob(r_k, r_v, layer=20, theta=500000.0):
    key = (r_k, r_v, layer, theta)
    if key not in _PROBS:
        _PROBS[key] = H.Problem(GEOM["D"], GEOM["H_q"], GEOM["H_kv"], GEOM["d_h"], r_k, r_v, theta=theta,
                                layer=layer)
    return _PROBS[key]


def _latents(prob, lens, layer):
    xs = [synth.hidden_states(int(L), prob.D, layer, chunk=200 + s).astype(np.float64) for s, L in enumerate(lens)]
    return H.oracle_latents(prob, xs)


def _run(sess, cache, q, n_splits=0):
    import torch
    b = q.shape[0]
    out = torch.zeros(b, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, n_splits=n_splits)
    assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
    assert sess.L.lorc_last_path(sess.ctx) == 2, "the tensor-core path was not taken"
    return out


@pytest.mark.parametrize("r_k,r_v,lens", [
    (96, 72, [1, 37, 300, 700]),          # rank tails below one 64-wide slice / one 128-row block
    (256, 256, [129, 128, 1000]),
    (928, 928, [513, 77]),                # largest rank of the 8B schedule: 14.5 slices, 7.25 blocks
    (1024, 1024, [260]),                  # full rank in latent form
])
def test_tc_decode_contiguous(r_k, r_v, lens):
    prob = _prob(r_k, r_v)
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    ck, cv = _latents(prob, lens, 20)
    cache, k, v, sl = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    for q_scale in (1.0, 64.0):
        q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 20, int(q_scale), q_scale).astype(np.float64)
        got = H.host_f64(_run(sess, cache, q))
        want = H.oracle_decode(prob, ck, cv, q)
        assert O.rel_l2_rows(got, want) <= TOL
    sess.close()


def test_tc_decode_large_batch_of_short_sequences():
    """More sequences than the score kernel caches lengths for, several 128-row blocks of output rows in the value
    up-projection, and contexts of one to three tiles."""
    prob = _prob(96, 72)
    b = 104
    lens = [int(v) for v in synth.ragged_lengths(b, 1, 300, base_seed=77)]
    n_max = max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    ck, cv = _latents(prob, lens, 20)
    cache, k, v, sl = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 20, 3, 8.0).astype(np.float64)
    got = H.host_f64(_run(sess, cache, q))
    want = H.oracle_decode(prob, ck, cv, q)
    assert O.rel_l2_rows(got, want) <= TOL
    sess.close()


def test_tc_decode_repeated_calls_are_bit_identical():
    """Back-to-back calls overlap their kernels' heads and tails (dependent launches), and the context shares of a
    column block are added by whichever share finishes last: neither may show in the result."""
    import torch
    prob = _prob(256, 256)
    lens = [1500, 700, 129]
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    ck, cv = _latents(prob, lens, 20)
    cache, k, v, sl = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    q = H.dev_bf16(synth.queries(b, GEOM["H_q"], GEOM["d_h"], 20, 5, 8.0).astype(np.float64))
    outs = [torch.zeros(b, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16, device="cuda") for _ in range(24)]
    for o in outs:                              # no synchronisation in between
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, q, o)
    torch.cuda.synchronize()
    assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
    for o in outs[1:]:
        assert torch.equal(o, outs[0])
    sess.close()


def test_tc_decode_matches_plain_kernels_and_split_counts():
    import torch
    prob = _prob(160, 224, layer=21)
    lens = [1500, 70, 640]
    b = len(lens)
    ck, cv = _latents(prob, lens, 21)
    q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 21, 0, 16.0).astype(np.float64)
    want = H.oracle_decode(prob, ck, cv, q)
    sess = H.Session(prob, max_pos=1536, batch=b)
    cache, k, v, sl = H.contiguous_cache(sess, b, 1536, lens, ck, cv)
    res = []
    for S in (0, 1, 2, 5, 12):
        res.append(H.host_f64(_run(sess, cache, q, n_splits=S)))
        assert O.rel_l2_rows(res[-1], want) <= TOL
    for r_ in res[1:]:
        assert O.rel_l2_rows(r_, res[0]) <= TOL        # same scores; p rounded against another max, output rounded to bf16
    sess.close()
    # the plain fp32 kernels agree with the tensor-core kernels within the bf16 tolerance
    dbg = H.Session(prob, max_pos=1536, batch=b, flags=1)
    cache, k, v, sl = H.contiguous_cache(dbg, b, 1536, lens, ck, cv)
    out = torch.zeros(b, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16, device="cuda")
    dbg.L.lorc_decode_attn(dbg.ctx, 0, cache, H.dev_bf16(q), out)
    assert dbg.L.lorc_last_path(dbg.ctx) == 1
    assert O.rel_l2_rows(res[0], H.host_f64(out)) <= TOL
    dbg.close()


def test_tc_decode_many_context_shares_with_64_query_heads():
    """Eight query heads per KV head, one sequence, one column block: the context is dealt over as many shares as it
    has tiles, more than one bulk-copy batch of the share reduction holds (four shares of 32 KiB), so the last share
    adds them up over several batches; forced share counts around the batch size as well."""
    import torch
    prob = H.Problem(GEOM["D"], 64, GEOM["H_kv"], GEOM["d_h"], 128, 128, theta=500000.0, layer=22)
    lens = [1500]
    ck, cv = _latents(prob, lens, 22)
    q = synth.queries(1, 64, GEOM["d_h"], 22, 0, 16.0).astype(np.float64)
    want = H.oracle_decode(prob, ck, cv, q)
    sess = H.Session(prob, max_pos=1536, batch=1)
    cache, k, v, sl = H.contiguous_cache(sess, 1, 1536, lens, ck, cv)
    for S in (0, 1, 4, 5, 9, 12):
        out = torch.zeros(1, 64, GEOM["d_h"], dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, n_splits=S)
        assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
        assert sess.L.lorc_last_path(sess.ctx) == 2, "the tensor-core path was not taken"
        assert O.rel_l2_rows(H.host_f64(out), want) <= TOL, S
    sess.close()


@pytest.mark.parametrize("page_size", [64, 16, 128])
def test_tc_decode_paged_and_page_permutation(page_size):
    import torch
    prob = _prob(96, 72, layer=22)
    lens = [200, 65, 64, 449]
    b = len(lens)
    sess = H.Session(prob, max_pos=512, batch=b)
    ck, cv = _latents(prob, lens, 22)
    q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 22, 0, 8.0).astype(np.float64)
    want = H.oracle_decode(prob, ck, cv, q)
    outs = []
    for order_seed in (11, 12):
        cache, k, v, sl, ptd, pt = H.paged_cache(sess, b, lens, page_size, order_seed, ck, cv)
        out = _run(sess, cache, q)
        assert O.rel_l2_rows(H.host_f64(out), want) <= TOL
        outs.append(out.clone())
    assert torch.equal(outs[0], outs[1])                # physical page order changes nothing
    cache, k, v, sl = H.contiguous_cache(sess, b, 512, lens, ck, cv)
    assert torch.equal(_run(sess, cache, q), outs[0])   # paged == contiguous, bit for bit
    sess.close()


def test_tc_ragged_batch_equals_each_sequence_alone_and_empty_sequence():
    import torch
    prob = _prob(96, 72, layer=23)
    lens = [17, 390, 128]
    sess = H.Session(prob, max_pos=512, batch=3)
    ck, cv = _latents(prob, lens, 23)
    q = synth.queries(3, GEOM["H_q"], GEOM["d_h"], 23, 0, 4.0)
    cache, k, v, sl = H.contiguous_cache(sess, 3, 512, lens, ck, cv)
    out = _run(sess, cache, q)
    for s in range(3):
        c1, k1, v1, sl1 = H.contiguous_cache(sess, 1, 512, [lens[s]], [ck[s]], [cv[s]])
        c1.max_seq_len = max(lens)
        o1 = _run(sess, c1, q[s:s + 1])
        assert torch.equal(o1[0], out[s])
    # an empty sequence gives zeros and status EMPTY; the others are unaffected
    sl[0] = 0
    o2 = torch.ones(3, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), o2)
    assert sess.L.lorc_sync_status(sess.ctx) == sess.L.LORC_ERR_EMPTY
    assert float(o2[0].abs().max()) == 0.0 and torch.equal(o2[1:], out[1:])
    # a page index outside the pool is reported, not dereferenced
    cache, k, v, sl, ptd, pt = H.paged_cache(sess, 3, lens, 64, 31, ck, cv)
    ptd[1, 2] = 10 ** 6
    sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), o2)
    assert sess.L.lorc_sync_status(sess.ctx) == sess.L.LORC_ERR_CAPACITY
    sess.close()


def test_tc_append_then_decode_chain_and_host_entry():
    import torch
    prob = _prob(96, 72, layer=24)
    b, N = 2, 300
    sess = H.Session(prob, max_pos=384, batch=b)
    xs = [synth.hidden_states(N + 1, prob.D, 24, chunk=300 + s).astype(np.float64) for s in range(b)]
    cache, k, v, sl = H.contiguous_cache(sess, b, 384, [N] * b)
    cache.max_seq_len = 384
    sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(np.stack([x[:N] for x in xs])), T=N)
    sl += 1
    q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 24, 0, 8.0)
    xh = torch.from_numpy(np.stack([x[N] for x in xs]).astype(np.float32)).to(torch.bfloat16).pin_memory()
    qh = torch.from_numpy(q).to(torch.bfloat16).pin_memory()
    oh = torch.zeros(b, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16).pin_memory()
    sess.L.lorc_decode_step_host(sess.ctx, 0, cache, xh, qh, oh)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    assert sess.L.lorc_last_path(sess.ctx) == 2
    ck, cv = H.oracle_latents(prob, xs)
    want = H.oracle_decode(prob, ck, cv, q.astype(np.float64))
    assert O.rel_l2_rows(H.host_f64(oh), want) <= TOL
    sess.close()


def test_tc_decode_one_context_serves_batches_of_different_sizes():
    """The library keeps one word per (sequence, head) for the softmax row maxima between calls, cleared by each call
    for the next and grown when a larger batch arrives: a small batch, a larger one and the small one again, on one
    context and one workspace, each against the oracle; queries of very different magnitudes in turn, so that a
    maximum left over from an earlier call would show."""
    import torch
    prob = _prob(256, 256)
    lens_small, lens_big = [300, 129], [64, 700, 1, 257, 513]
    n_max = 720
    sess = H.Session(prob, max_pos=n_max, batch=len(lens_big))
    for it, (lens, q_scale) in enumerate([(lens_small, 64.0), (lens_big, 1.0), (lens_small, 0.25), (lens_big, 64.0)]):
        b = len(lens)
        ck, cv = _latents(prob, lens, 20)
        cache, k, v, sl = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
        q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 20, 30 + it, q_scale).astype(np.float64)
        got = H.host_f64(_run(sess, cache, q))
        want = H.oracle_decode(prob, ck, cv, q)
        assert O.rel_l2_rows(got, want) <= TOL, (it, O.rel_l2_rows(got, want))
    sess.close()


# ------------------------------------------------------------------- uncompressed reference mode, 128-wide heads
@pytest.mark.parametrize("H_q,lens,paged", [
    (32, [700, 64, 1, 129], False),          # G = 4
    (64, [300, 517], False),                 # G = 8
    (32, [450, 33, 200], True),              # 64-token pages in a random physical order
])
def test_full_rank_mode_streaming_kernel(H_q, lens, paged):
    """Ordinary KV cache (keys stored rotated): the streaming decode kernel against textbook attention over the
    uncompressed weights, with several context-split counts."""
    import torch
    D, H_kv, d_h = 1024, 8, 128
    prob = H.Problem(D, H_q, H_kv, d_h, 64, 64, theta=500000.0, layer=31)
    b, n_max = len(lens), max(lens) + 5
    sess = H.Session(prob, max_pos=n_max, batch=b, mode=1)
    xs = [synth.hidden_states(n_max, D, 31, chunk=300 + s).astype(np.float64) for s in range(b)]
    if paged:
        cache, k, v, sl, ptd, pt = H.paged_cache(sess, b, [n_max] * b, 64, order_seed=5)
    else:
        cache, k, v, sl = H.contiguous_cache(sess, b, n_max, [n_max] * b)
    sess.L.lorc_append(sess.ctx, 0, cache, H.dev_bf16(np.stack(xs)), T=n_max)
    assert sess.L.lorc_last_path(sess.ctx) == 2, "the mma cache-write kernel was not taken"
    if not paged:
        # the cache holds the rotated key projections and the value projections, each rounded once
        Kr = O.rope((xs[0] @ prob.W_k).reshape(-1, H_kv, d_h), np.arange(n_max)[:, None], prob.theta).reshape(-1, prob.n)
        assert np.all(np.abs(H.host_f64(k[0]) - Kr) <= H.bf16_ulp(Kr) + 1e-6)
        Vp = xs[0] @ prob.W_v
        assert np.all(np.abs(H.host_f64(v[0]) - Vp) <= H.bf16_ulp(Vp) + 1e-6)
    sl[:] = torch.tensor(lens, dtype=torch.int32)
    q = synth.queries(b, H_q, d_h, 31, 1, 8.0).astype(np.float64)
    want = [O.decode_attn_full(xs[s][:lens[s]], prob.W_k, prob.W_v, q[s], H_kv, prob.theta) for s in range(b)]
    outs = []
    for n_splits in (0, 1, 3):
        out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, n_splits=n_splits)
        assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
        assert sess.L.lorc_last_path(sess.ctx) == 3, "the streaming kernel of the uncompressed mode was not taken"
        got = H.host_f64(out)
        for s in range(b):
            assert O.rel_l2_rows(got[s], want[s]) <= TOL, (n_splits, s, O.rel_l2_rows(got[s], want[s]))
        outs.append(got)
    sess.close()


# --------------------------------------------------------------- no rotation: the absorbed score path
@pytest.mark.parametrize("r_k,r_v,lens,paged", [
    (96, 72, [1, 37, 300, 700], False),
    (256, 256, [129, 128, 1000], True),
    (928, 928, [513, 77], False),
])
def test_tc_decode_without_rotation_uses_the_absorbed_scores(r_k, r_v, lens, paged):
    """LORC_ROPE_NONE: s = (B_K q) . c (Sec. 3.1, the W_q' equation) on the tensor cores, against the oracle, which
    reconstructs the keys explicitly and applies no rotation."""
    key = (r_k, r_v, "none")
    if key not in _PROBS:
        _PROBS[key] = H.Problem(GEOM["D"], GEOM["H_q"], GEOM["H_kv"], GEOM["d_h"], r_k, r_v, theta=500000.0, layer=21,
                                style=H.ROPE_NONE)
    prob = _PROBS[key]
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    ck, cv = _latents(prob, lens, 21)
    # (the descriptor only holds addresses: the tensors behind it must stay alive)
    if paged:
        held = H.paged_cache(sess, b, lens, 64, order_seed=5, k_rows=ck, v_rows=cv)
    else:
        held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    cache = held[0]
    worst = 0.0
    for q_scale in (1.0, 64.0):
        q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 21, int(q_scale), q_scale).astype(np.float64)
        got = H.host_f64(_run(sess, cache, q))
        want = H.oracle_decode(prob, ck, cv, q)
        H.assert_rows_close(got, want, TOL, (r_k, q_scale))
        worst = max(worst, O.rel_l2_rows(got, want))
    print(f"\n[no rotation] r_k {r_k}: max relative L2 row error {worst:.2e}")
    sess.close()


@pytest.mark.parametrize("style", [0, H.ROPE_NONE])
def test_tc_latent_output_entry(style):
    """lorc_decode_attn_latent_out on the tensor-core path: the normalised latent output [b, H_q, r_v] against the
    oracle, and its product with B_V against lorc_decode_attn's result."""
    import torch
    r_k, r_v, lens = 256, 200, [700, 130, 1]
    prob = H.Problem(GEOM["D"], GEOM["H_q"], GEOM["H_kv"], GEOM["d_h"], r_k, r_v, theta=500000.0, layer=22, style=style)
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    ck, cv = _latents(prob, lens, 22)
    held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    q = synth.queries(b, GEOM["H_q"], GEOM["d_h"], 22, 1, 8.0).astype(np.float64)
    o_lat = torch.zeros(b, GEOM["H_q"], r_v, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn_latent_out(sess.ctx, 0, held[0], H.dev_bf16(q), o_lat)
    assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
    assert sess.L.lorc_last_path(sess.ctx) == 2
    got = H.host_f64(o_lat)
    for s in range(b):
        want = O.decode_attn_latent_out(ck[s], cv[s], prob.B_k, q[s], GEOM["H_kv"], prob.theta,
                                        use_rope=style != H.ROPE_NONE)
        assert O.rel_l2_rows(got[s], want) <= TOL
    # the ordinary entry afterwards (the row maxima were left empty) agrees with o_lat . B_V
    out = H.host_f64(_run(sess, held[0], q))
    G = GEOM["H_q"] // GEOM["H_kv"]
    for h in range(GEOM["H_q"]):
        g = h // G
        proj = got[:, h, :] @ prob.B_v[:, g * 128:(g + 1) * 128]
        assert O.rel_l2_rows(out[:, h, :], proj) <= TOL
    sess.close()
