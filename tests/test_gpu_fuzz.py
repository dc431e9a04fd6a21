"""Seeded random shapes on the tensor-core path against the plain fp32 kernels of the same library (which the other
tests hold against the oracle): ranks that are not multiples of 64 or 128, ragged batches with empty and one-token
sequences, contiguous and paged caches with every page size, both group sizes, explicit context shares, decode and
the latent-output entry.  Every case also runs on the oracle for its first sequence."""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu
TOL = 1e-2
_FACTORS = {}


def _problem(H_q, H_kv, r_k, r_v, layer):
    """Factors cut from one set of generators per geometry (the generators are the expensive part)."""
    key = (H_q, H_kv, layer)
    if key not in _FACTORS:
        n = H_kv * 128
        _FACTORS[key] = H.Problem(max(1024, n), H_q, H_kv, 128, n, n, theta=500000.0, layer=layer)
    full = _FACTORS[key]
    prob = H.Problem.__new__(H.Problem)
    prob.__dict__.update(full.__dict__)
    prob.r_k, prob.r_v = r_k, r_v
    prob.A_k, prob.B_k = full.A_k[:, :r_k].copy(), full.B_k[:r_k].copy()
    prob.A_v, prob.B_v = full.A_v[:, :r_v].copy(), full.B_v[:r_v].copy()
    return prob


@pytest.mark.parametrize("seed", range(24))
def test_random_shape_tensor_core_path_equals_plain_path(seed):
    import torch
    rng = np.random.default_rng(1000 + seed)
    H_q, H_kv = [(32, 8), (64, 8), (32, 4), (64, 16)][seed % 4]
    r_max = min(1024, H_kv * 128) // 8
    r_k = int(rng.integers(1, r_max + 1)) * 8
    r_v = int(rng.integers(1, r_max + 1)) * 8
    b = int(rng.integers(1, 7))
    lens = [int(x) for x in rng.integers(1, 900, size=b)]
    if seed % 5 == 0:
        lens[0] = 1
    if seed % 7 == 3 and b > 1:
        lens[-1] = 0                      # an empty sequence: zeros, status EMPTY
    paged = seed % 3 == 1
    page_size = [16, 32, 64, 128][seed % 4]
    n_splits = [0, 0, 1, 3, 7][seed % 5]
    latent_out = seed % 6 == 2
    prob = _problem(H_q, H_kv, r_k, r_v, 40 + seed % 4)
    n_max = max(lens) + int(rng.integers(0, 5))
    n_max = max(n_max, 1)
    L = H.lib()
    ck = [synth.to_bf16_exact(rng.standard_normal((n, r_k)) * (np.arange(1, r_k + 1) ** -0.8)) for n in lens]
    cv = [synth.to_bf16_exact(rng.standard_normal((n, r_v)) * (np.arange(1, r_v + 1) ** -0.8)) for n in lens]
    q = synth.queries(b, H_q, 128, 40, seed, [1.0, 8.0, 64.0][seed % 3]).astype(np.float64)
    outs = []
    for flags, path in ((0, 2), (L.LORC_FLAG_DEBUG_FP32, 1)):
        sess = H.Session(prob, max_pos=n_max, batch=b, flags=flags)
        if paged:
            held = H.paged_cache(sess, b, lens, page_size, order_seed=seed, k_rows=ck, v_rows=cv)
        else:
            held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
        width = r_v if latent_out else 128
        out = torch.full((b, H_q, width), 5.0, dtype=torch.bfloat16, device="cuda")
        if latent_out:
            L.lorc_decode_attn_latent_out(sess.ctx, 0, held[0], H.dev_bf16(q), out, n_splits=n_splits)
        else:
            L.lorc_decode_attn(sess.ctx, 0, held[0], H.dev_bf16(q), out, n_splits=n_splits)
        rc = L.lorc_sync_status(sess.ctx)
        assert rc == (L.LORC_ERR_EMPTY if 0 in lens else 0), (rc, L.lorc_last_error(sess.ctx))
        assert L.lorc_last_path(sess.ctx) == path
        outs.append(H.host_f64(out))
        sess.close()
    tc, plain = outs
    live = [s for s in range(b) if lens[s] > 0]
    assert O.rel_l2_rows(tc[live], plain[live]) <= TOL, (seed, r_k, r_v, lens, paged, page_size, n_splits)
    for s in range(b):
        if lens[s] == 0:
            assert np.all(tc[s] == 0.0) and np.all(plain[s] == 0.0)
    s0 = live[0]
    if latent_out:
        want = O.decode_attn_latent_out(ck[s0], cv[s0], prob.B_k, q[s0], H_kv, prob.theta)
    else:
        want = O.decode_attn_latent(ck[s0], cv[s0], prob.B_k, prob.B_v, q[s0], H_kv, prob.theta)
    assert O.rel_l2_rows(tc[s0], want) <= TOL


@pytest.mark.parametrize("seed", range(10))
def test_random_prompt_chunk_tensor_core_path_equals_plain_path(seed):
    """Prompt chunks of random length over random prefixes (every sequence holds at least the chunk)."""
    import torch
    rng = np.random.default_rng(2000 + seed)
    H_q, H_kv = [(32, 8), (64, 8), (32, 4)][seed % 3]
    r_max = min(1024, H_kv * 128) // 8
    r_k, r_v = int(rng.integers(1, r_max + 1)) * 8, int(rng.integers(1, r_max + 1)) * 8
    b = int(rng.integers(1, 4))
    T = int(rng.integers(1, 200))
    lens = [T + int(x) for x in rng.integers(0, 500, size=b)]
    if seed % 4 == 0:
        lens[0] = T                       # no prefix: the chunk is the whole sequence
    paged = seed % 2 == 1
    page_size = [16, 32, 64, 128][seed % 4]
    prob = _problem(H_q, H_kv, r_k, r_v, 40 + seed % 4)
    n_max = max(lens) + 2
    L = H.lib()
    ck = [synth.to_bf16_exact(rng.standard_normal((n, r_k)) * (np.arange(1, r_k + 1) ** -0.8)) for n in lens]
    cv = [synth.to_bf16_exact(rng.standard_normal((n, r_v)) * (np.arange(1, r_v + 1) ** -0.8)) for n in lens]
    q = synth.to_bf16_exact([1.0, 8.0][seed % 2] * synth.gaussian((b, T, H_q, 128), 41, seed)).astype(np.float64)
    outs = []
    for flags, path in ((0, 2), (L.LORC_FLAG_DEBUG_FP32, 1)):
        sess = H.Session(prob, max_pos=n_max, batch=b, flags=flags)
        if paged:
            held = H.paged_cache(sess, b, lens, page_size, order_seed=seed, k_rows=ck, v_rows=cv)
        else:
            held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
        ws = torch.zeros(L.lorc_prefill_workspace_bytes(sess.ctx, b, max(lens), T), dtype=torch.uint8, device="cuda")
        L.lorc_set_workspace(sess.ctx, ws)
        out = torch.full((b, T, H_q, 128), 5.0, dtype=torch.bfloat16, device="cuda")
        L.lorc_prefill_attn(sess.ctx, 0, held[0], H.dev_bf16(q), out, T)
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == path
        outs.append(H.host_f64(out))
        sess.close()
    assert O.rel_l2_rows(outs[0], outs[1]) <= TOL, (seed, r_k, r_v, lens, T, paged, page_size)
    # the oracle on the last query of the first sequence (it sees the whole cache) and on its first query
    want_last = O.decode_attn_latent(ck[0], cv[0], prob.B_k, prob.B_v, q[0, T - 1], H_kv, prob.theta)
    assert O.rel_l2_rows(outs[0][0, T - 1], want_last) <= TOL
    n_first = lens[0] - T + 1
    want_first = O.decode_attn_latent(ck[0][:n_first], cv[0][:n_first], prob.B_k, prob.B_v, q[0, 0], H_kv, prob.theta)
    assert O.rel_l2_rows(outs[0][0, 0], want_first) <= TOL


@pytest.mark.parametrize("seed", range(8))
def test_random_context_cuts_merge_to_the_whole(seed):
    """Context shards cut at arbitrary positions (not tile multiples), some of them empty: merged result against the
    unsharded call and the oracle."""
    import torch
    rng = np.random.default_rng(3000 + seed)
    H_q, H_kv = [(32, 8), (64, 8)][seed % 2]
    r_k, r_v = int(rng.integers(1, 129)) * 8, int(rng.integers(1, 129)) * 8
    b = int(rng.integers(1, 4))
    lens = [int(x) for x in rng.integers(1, 700, size=b)]
    world = int(rng.integers(2, 5))
    prob = _problem(H_q, H_kv, r_k, r_v, 40 + seed % 4)
    n_max = max(lens) + 1
    L = H.lib()
    ck = [synth.to_bf16_exact(rng.standard_normal((n, r_k)) * (np.arange(1, r_k + 1) ** -0.8)) for n in lens]
    cv = [synth.to_bf16_exact(rng.standard_normal((n, r_v)) * (np.arange(1, r_v + 1) ** -0.8)) for n in lens]
    q = synth.queries(b, H_q, 128, 42, seed, 8.0).astype(np.float64)
    cuts = [sorted([0, n] + [int(x) for x in rng.integers(0, n + 1, size=world - 1)]) for n in lens]
    sess = H.Session(prob, max_pos=n_max, batch=b)
    qd = H.dev_bf16(q)
    q_pos = torch.tensor([n - 1 for n in lens], dtype=torch.int32, device="cuda")
    outs = torch.zeros(world, b, H_q, 128, dtype=torch.bfloat16, device="cuda")
    mls = torch.zeros(world, b, H_q, 2, dtype=torch.float32, device="cuda")
    keep = []
    for r in range(world):
        p0 = [cuts[s][r] for s in range(b)]
        cnt = [cuts[s][r + 1] - cuts[s][r] for s in range(b)]
        held = H.contiguous_cache(sess, b, n_max, cnt, [ck[s][p0[s]:p0[s] + cnt[s]] for s in range(b)],
                                  [cv[s][p0[s]:p0[s] + cnt[s]] for s in range(b)])
        keep.append(held)
        L.lorc_decode_attn_shard(sess.ctx, 0, held[0], qd, torch.tensor(p0, dtype=torch.int32, device="cuda"), q_pos,
                                 outs[r], mls[r])
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == 2
    merged = torch.zeros(b, H_q, 128, dtype=torch.bfloat16, device="cuda")
    L.lorc_merge_shards(sess.ctx, world, outs, mls, merged, b)
    assert L.lorc_sync_status(sess.ctx) == 0
    want = H.oracle_decode(prob, ck, cv, q)
    assert O.rel_l2_rows(H.host_f64(merged), want) <= 1.5 * TOL, (seed, cuts)
    sess.close()


@pytest.mark.parametrize("seed", range(10))
def test_random_cache_write_equals_oracle_rows(seed):
    """lorc_append at random token counts (one token: the decode kernel; 128 and more per launch: the tcgen05 GEMM), ranks,
    prefixes and cache layouts: every written row within one bf16 ulp of the exactly rounded latent, rows before and
    after the written range untouched."""
    import torch
    rng = np.random.default_rng(4000 + seed)
    H_q, H_kv = [(32, 8), (64, 8)][seed % 2]
    r_k, r_v = int(rng.integers(1, 129)) * 8, int(rng.integers(1, 129)) * 8
    b = int(rng.integers(1, 5))
    T = [1, 1, 3, 16, 40, 128, 130, 200, 257, 64][seed]
    prefix = [int(x) for x in rng.integers(0, 300, size=b)]
    lens = [p + T for p in prefix]
    paged = seed % 3 == 1
    page_size = [16, 32, 64, 128][seed % 4]
    prob = _problem(H_q, H_kv, r_k, r_v, 40 + seed % 4)
    n_max = max(lens) + 3
    L = H.lib()
    sess = H.Session(prob, max_pos=n_max, batch=b)
    x = np.stack([synth.hidden_states(T, prob.D, 44, chunk=10 * seed + s) for s in range(b)]).astype(np.float64)
    if paged:
        held = H.paged_cache(sess, b, lens, page_size, order_seed=seed)
    else:
        held = H.contiguous_cache(sess, b, n_max, lens)
    held[1].fill_(3.0)                   # whatever is not written must keep this
    held[2].fill_(3.0)
    L.lorc_append(sess.ctx, 0, held[0], H.dev_bf16(x), T=T)
    assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
    kk, vv = H.host_f64(held[1]), H.host_f64(held[2])
    for s in range(b):
        want_k = O.append_latent_bf16(x[s], prob.A_k)
        want_v = O.append_latent_bf16(x[s], prob.A_v)
        exact_k, exact_v = O.append_latent(x[s], prob.A_k), O.append_latent(x[s], prob.A_v)
        for t in range(T):
            pos = prefix[s] + t
            if paged:
                page = int(held[5][s, pos // page_size])
                row_k, row_v = kk[page, pos % page_size], vv[page, pos % page_size]
            else:
                row_k, row_v = kk[s, pos], vv[s, pos]
            # one ulp of the rounded value, plus the fp32 accumulation bound where the terms cancel
            for got, want, exact, A in ((row_k, want_k[t], exact_k[t], prob.A_k), (row_v, want_v[t], exact_v[t], prob.A_v)):
                slack = 2.0 ** -16 * (np.abs(x[s][t])[:, None] * np.abs(A)).sum(0)
                assert np.all(np.abs(got - want) <= H.bf16_ulp(want) + slack), (seed, s, t)
        if not paged:
            assert np.all(kk[s, :prefix[s]] == 3.0) and np.all(kk[s, lens[s]:] == 3.0)
            assert np.all(vv[s, :prefix[s]] == 3.0) and np.all(vv[s, lens[s]:] == 3.0)
    sess.close()
