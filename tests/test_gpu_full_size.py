"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The workload object of bench.py is built for a whole configuration (all sequences, the full context, the
library's own prefill), one decode step is launched call by call and a second one as a CUDA-graph replay, exactly
as the benchmark does.  The oracle cannot redo all of that, so it redoes sampled (layer, sequence) outputs one by
one.  Two kinds of sample:
  chain   from the seeded inputs alone: the oracle derives the factors from the weight generators, the latents
          from the hidden states (Sec. 3.1) and the attention output from those (Sec. 3.3 with the position embedding
          applied at attention time); nothing the CUDA path produced enters it, and the cache rows the device wrote
          are checked against the exactly rounded latents on the way;
  kernel  the oracle reads the cache rows back from the device (bf16 values, exact in fp64) and redoes the attention
          over them: the same check of the attention kernels at a fraction of the cost.
Every sampled (layer, sequence) is attended with the benchmark's query (scale 8) and again, on the cache rows the
device holds, with queries of scale 1 (near-uniform softmax) and 64 (peaked softmax, where rotation or position errors
show).
Each test prints the largest error it saw.
"""
import os
import sys

import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TOL = 1e-2          # max relative L2 error of a (sequence, head) output row, bf16 path
CHUNK = 512         # prompt chunk of the benchmark's prefill


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _cfg2_samples():
    chain = [(l, (5 * l + 3) % 16) for l in range(32)]
    kernel = [(l, (11 * l + 8) % 16) for l in range(32)]
    return chain, kernel


CASES = [
    # configuration, layers of it that are built, chain samples, kernel samples (layer index in the built list, sequence)
    ("cfg2_8b_progressive", list(range(32))) + _cfg2_samples(),
    ("cfg3_8b_long", [0], [(0, 2)], [(0, 0)]),
    # ranks 864, 608 and 352 of the 70B schedule (8 query heads per KV head)
    ("cfg4_70b_progressive", [0, 38, 79], [(0, 5), (2, 1)], [(1, 3), (2, 6)]),
]


def _factors(shape, lid, r, device):
    from workloads import device as wdev
    fac = {}
    for which in ("k", "v"):
        U, sg, V = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, lid, which, device)
        A, B = O.factors_from_generators(_f64(U), _f64(sg), _f64(V), r)
        fac[which] = (synth.to_bf16_exact(A), synth.to_bf16_exact(B))
        del U, V
    return fac


def _attend_scales(L, wl, l, cache_rows, fac, shape, seqs, worst):
    """Attention of layer l with queries of scale 1 and 64 on the cache as it stands; checks sequences `seqs`."""
    import torch
    from workloads import device as wdev
    for scale in (1.0, 64.0):
        q = wdev.queries((shape.batch, shape.n_q_heads, shape.d_head), wl.layer_ids[l], 900 + int(scale), wl.out.device, scale)
        out = torch.zeros_like(wl.out[l])
        L.lorc_decode_attn(wl.ctx, l, wl.caches[l], q, out)
        torch.cuda.synchronize()
        assert L.lorc_sync_status(wl.ctx) == 0, L.lorc_last_error(wl.ctx)
        for s in seqs:
            ck, cv = cache_rows[s]
            want = O.decode_attn_latent(ck, cv, fac["k"][1], fac["v"][1], _f64(q[s]), shape.n_kv_heads, shape.rope_theta)
            got = _f64(out[s])
            helpers.assert_rows_close(got, want, TOL, (shape.name, l, s, scale))
            worst[scale] = max(worst.get(scale, 0.0), O.rel_l2_rows(got, want))


@pytest.mark.gpu
@pytest.mark.parametrize("name,layer_ids,chain,kernel", CASES, ids=[c[0] for c in CASES])
def test_sampled_outputs_at_full_size(name, layer_ids, chain, kernel):
    import torch
    sys.path.insert(0, ROOT)
    import bench
    from workloads import device as wdev
    L = helpers.lib()
    shape = synth.CONFIGS[name]
    device = torch.device("cuda", 0)
    wl = bench.Workload(L, shape, len(layer_ids), 4, device, 0, layer_ids=layer_ids)
    wl.step()                     # call by call
    torch.cuda.synchronize()
    wl.capture()
    wl.step_graph()               # the graph replay the benchmark times
    torch.cuda.synchronize()
    assert L.lorc_sync_status(wl.ctx) == 0, L.lorc_last_error(wl.ctx)
    assert L.lorc_last_path(wl.ctx) == 2          # tensor-core kernels, not the plain ones
    steps_done = 2
    N = shape.context + steps_done
    assert int(wl.seq_lens[0]) == N
    worst = {}
    by_layer = {}
    for (l, s) in chain:
        by_layer.setdefault(l, ([], []))[0].append(s)
    for (l, s) in kernel:
        by_layer.setdefault(l, ([], []))[1].append(s)
    for l, (chain_s, kernel_s) in sorted(by_layer.items()):
        lid, r = layer_ids[l], shape.ranks[layer_ids[l]]
        # factors from the generators of the synthetic weights, rounded to bf16 as the library holds them
        fac = _factors(shape, lid, r, device)
        rows = {}
        for s in chain_s:
            # hidden states of this sequence: the prefill chunks, then the decode steps
            xs = [_f64(wdev.hidden_states((shape.batch, min(CHUNK, shape.context - c0), shape.d_model), lid, c0 // CHUNK,
                                          device)[s]) for c0 in range(0, shape.context, CHUNK)]
            xs += [_f64(wl.x[l][i][s])[None, :] for i in range(steps_done)]
            X = np.concatenate(xs, axis=0)
            assert X.shape == (N, shape.d_model)
            ck = O.append_latent_bf16(X, fac["k"][0])
            cv = O.append_latent_bf16(X, fac["v"][0])
            # Cache write: the device's latents against the exactly rounded ones.  Bound: one bf16 ulp of the exact
            # latent (the final rounding may fall either way) plus the fp32 accumulation error of a D-term dot product,
            # taken as 2^-16 of sum_i |x_i A_ij| (between the typical sqrt(D) 2^-24 and the worst case D 2^-24 for
            # D = 4096 ... 8192); the second term only matters where the terms cancel to a latent far smaller than
            # themselves.
            for ref, dev, A in ((ck, wl.keep[l][0], fac["k"][0]), (cv, wl.keep[l][1], fac["v"][0])):
                got = _f64(dev[s, :N])
                err = np.abs(got - ref)
                bound = helpers.bf16_ulp(ref) + 2.0 ** -16 * (np.abs(X) @ np.abs(A))
                assert np.all(err <= bound), float((err / bound).max())
                assert np.mean(err > 0) < 0.02          # a different last bit only where fp32 and fp64 sums straddle a tie
                worst["cache write, error / bound"] = max(worst.get("cache write, error / bound", 0.0), float((err / bound).max()))
                worst["cache write, fraction of entries off by an ulp"] = max(
                    worst.get("cache write, fraction of entries off by an ulp", 0.0), float(np.mean(err > 0)))
            rows[s] = (ck, cv)
        for s in kernel_s:
            rows[s] = (_f64(wl.keep[l][0][s, :N]), _f64(wl.keep[l][1][s, :N]))
        # the benchmark's own step (query scale 8)
        for s in sorted(rows):
            ck, cv = rows[s]
            q = _f64(wl.q[l][steps_done - 1][s])
            want = O.decode_attn_latent(ck, cv, fac["k"][1], fac["v"][1], q, shape.n_kv_heads, shape.rope_theta)
            got = _f64(wl.out[l, s])
            helpers.assert_rows_close(got, want, TOL, (name, l, s, 8.0))
            worst[8.0] = max(worst.get(8.0, 0.0), O.rel_l2_rows(got, want))
        # The other two query scales test the attention kernels, so they run on the rows the device holds (read back;
        # bf16 values are exact in fp64): a peaked softmax (scale 64) turns a last-bit difference in one large latent
        # coordinate into a visible change of the output, which is a property of the cache write's rounding, checked
        # above, not of the attention.
        held_rows = {s: (_f64(wl.keep[l][0][s, :N]), _f64(wl.keep[l][1][s, :N])) for s in rows}
        _attend_scales(L, wl, l, held_rows, fac, shape, sorted(rows), worst)
    print(f"\n[full size] {name}: layers {sorted(set(layer_ids[l] for l in by_layer))}, "
          f"{len(chain)} chain + {len(kernel)} kernel samples; max relative L2 row error by query scale "
          + ", ".join(f"{k}: {v:.2e}" for k, v in sorted(worst.items(), key=lambda kv: str(kv[0]))))
    wl.close()
    torch.cuda.empty_cache()


RAGGED = ["cfg5_ragged_r128", "cfg5_ragged_r256", "cfg5_ragged_r384", "cfg5_ragged_r1024"]


def _append_through_pages(L, sess, prob, k, v, sl, ptd, s, x, page_size, max_pages, n_pages):
    """Write sequence s of a paged cache with lorc_append, in chunks, through a one-sequence view of the cache."""
    import torch
    n = x.shape[0]
    view_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    cache1 = L.make_cache(k, v, view_len, 1, int(max_pages * page_size), page_table=ptd[s:s + 1], page_size=page_size,
                          max_pages_per_seq=max_pages, n_pages=n_pages)
    done = 0
    while done < n:
        T = min(CHUNK, n - done)
        view_len.fill_(done + T)
        L.lorc_append(sess.ctx, 0, cache1, helpers.dev_bf16(x[done:done + T])[None], T=T)
        done += T
    torch.cuda.synchronize()


@pytest.mark.gpu
@pytest.mark.parametrize("name", RAGGED)
def test_ragged_paged_batch_at_full_size(name):
    """64 sequences of 512 ... 16384 tokens in 64-token pages scattered over the pool.  Most cache rows are seeded;
    the shortest sequence and one of middle length are written by lorc_append through the page table from seeded
    hidden states.  The shortest, the longest and two more sequences are checked against the oracle, which reads the
    same cache rows through the same page table (and, for the appended ones, also derives them itself)."""
    import torch
    from workloads import device as wdev
    L = helpers.lib()
    shape = synth.CONFIGS[name]
    device = torch.device("cuda", 0)
    r = shape.ranks[0]
    prob = helpers.Problem(shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.d_head, r, r, theta=shape.rope_theta,
                           p=shape.sigma_p)
    lens = synth.ragged_lengths(shape.batch, shape.ragged[0], shape.ragged[1])
    sess = helpers.Session(prob, int(lens.max()) + 64, shape.batch)
    cache, k, v, sl, ptd, pt = helpers.paged_cache(sess, shape.batch, lens, shape.page_size, order_seed=11)
    k.copy_(wdev.latents(tuple(k.shape), shape.sigma_p, 0, "k", device))
    v.copy_(wdev.latents(tuple(v.shape), shape.sigma_p, 0, "v", device))
    order = np.argsort(lens)
    picks = [int(order[0]), int(order[-1]), int(order[len(order) // 3]), int(order[2 * len(order) // 3])]
    appended = {}
    for s in (picks[0], picks[2]):
        x = synth.hidden_states(int(lens[s]), shape.d_model, 0, chunk=700 + s).astype(np.float64)
        _append_through_pages(L, sess, prob, k, v, sl, ptd, s, x, shape.page_size, pt.shape[1], k.shape[0])
        appended[s] = x
    assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
    ps = shape.page_size
    worst = {}
    for scale in (1.0, 8.0, 64.0):
        q = wdev.queries((shape.batch, shape.n_q_heads, shape.d_head), 0, int(scale), device, scale)
        out = torch.zeros(shape.batch, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
        L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
        torch.cuda.synchronize()
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == 2
        got_all = _f64(out)
        assert np.all(np.isfinite(got_all))
        for s in picks:
            n = int(lens[s])
            pages = torch.tensor(pt[s, :(n + ps - 1) // ps].astype(np.int64), device=device)
            ck = _f64(k[pages].reshape(-1, r)[:n])
            cv = _f64(v[pages].reshape(-1, r)[:n])
            if s in appended and scale == 8.0:
                # the rows lorc_append wrote through the page table against the oracle's own latents
                for got_rows, A in ((ck, prob.A_k), (cv, prob.A_v)):
                    ref = O.append_latent_bf16(appended[s], A)
                    err = np.abs(got_rows - ref)
                    bound = helpers.bf16_ulp(ref) + 2.0 ** -16 * (np.abs(appended[s]) @ np.abs(A))
                    assert np.all(err <= bound), float((err / bound).max())
            want = O.decode_attn_latent(ck, cv, prob.B_k, prob.B_v, _f64(q[s]), shape.n_kv_heads, shape.rope_theta)
            helpers.assert_rows_close(got_all[s], want, TOL, (name, s, n, scale))
            worst[scale] = max(worst.get(scale, 0.0), O.rel_l2_rows(got_all[s], want))
    print(f"\n[full size] {name}: sequences {picks} (lengths {[int(lens[s]) for s in picks]}); max relative L2 row error "
          "by query scale " + ", ".join(f"{k_}: {v_:.2e}" for k_, v_ in sorted(worst.items())))
    sess.close()
    del k, v
    torch.cuda.empty_cache()


@pytest.mark.gpu
def test_ragged_paged_batch_uncompressed_mode():
    """The uncompressed reference mode on the ragged paged batch (the 16 first sequences of it, so that whole keys and
    values fit next to everything else): keys and values written by lorc_append through the page table for two
    sequences, seeded for the rest; outputs against the oracle's textbook attention over the same cache rows."""
    import torch
    from workloads import device as wdev
    L = helpers.lib()
    shape = synth.CONFIGS["cfg5_ragged_r256"]
    device = torch.device("cuda", 0)
    b = 16
    prob = helpers.Problem(shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.n, shape.n,
                           theta=shape.rope_theta, p=shape.sigma_p)
    lens = synth.ragged_lengths(shape.batch, shape.ragged[0], shape.ragged[1])[:b]
    sess = helpers.Session(prob, int(lens.max()) + 64, b, mode=L.LORC_MODE_FULL)
    cache, k, v, sl, ptd, pt = helpers.paged_cache(sess, b, lens, shape.page_size, order_seed=12)
    n = shape.n
    k.copy_(wdev.latents(tuple(k.shape), 0.0, 0, "k", device))
    v.copy_(wdev.latents(tuple(v.shape), 0.0, 0, "v", device))
    order = np.argsort(lens)
    picks = [int(order[0]), int(order[-1]), int(order[b // 2])]
    s_app = picks[0]
    x = synth.hidden_states(int(lens[s_app]), shape.d_model, 0, chunk=800).astype(np.float64)
    _append_through_pages(L, sess, prob, k, v, sl, ptd, s_app, x, shape.page_size, pt.shape[1], k.shape[0])
    assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
    ps = shape.page_size
    worst = {}
    for scale in (1.0, 64.0):
        q = wdev.queries((b, shape.n_q_heads, shape.d_head), 0, int(scale), device, scale)
        out = torch.zeros(b, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
        L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
        torch.cuda.synchronize()
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == 3
        got_all = _f64(out)
        for s in picks:
            m = int(lens[s])
            pages = torch.tensor(pt[s, :(m + ps - 1) // ps].astype(np.int64), device=device)
            kk = _f64(k[pages].reshape(-1, n)[:m])
            vv = _f64(v[pages].reshape(-1, n)[:m])
            # cached keys are already rotated: textbook attention with the query rotated at its position
            want = O.decode_attn_cached_kv(kk.reshape(m, shape.n_kv_heads, shape.d_head),
                                           vv.reshape(m, shape.n_kv_heads, shape.d_head), _f64(q[s]), shape.rope_theta)
            if s == s_app and scale == 1.0:
                # the rows lorc_append wrote in this mode: keys rotated at their positions, values as they are
                k_ref = O.rope((x @ prob.W_k).reshape(m, shape.n_kv_heads, shape.d_head), np.arange(m)[:, None],
                               shape.rope_theta).reshape(m, n)
                v_ref = x @ prob.W_v
                for got_rows, ref, W in ((kk, k_ref, prob.W_k), (vv, v_ref, prob.W_v)):
                    bound = 2.0 * helpers.bf16_ulp(ref) + 2.0 ** -15 * (np.abs(x) @ np.abs(W))
                    assert np.all(np.abs(got_rows - O.bf16_round(ref)) <= bound)
            helpers.assert_rows_close(got_all[s], want, TOL, ("full", s, m, scale))
            worst[scale] = max(worst.get(scale, 0.0), O.rel_l2_rows(got_all[s], want))
    print(f"\n[full size] uncompressed mode, ragged paged: sequences {picks}; max relative L2 row error by query scale "
          + ", ".join(f"{k_}: {v_:.2e}" for k_, v_ in sorted(worst.items())))
    sess.close()
    del k, v
    torch.cuda.empty_cache()


@pytest.mark.gpu
@pytest.mark.parametrize("name,layer_ids,T,picks", [
    # the last 1024 tokens of the 4096-token prompts as the chunk; ranks 928 and 416
    ("cfg2_8b_progressive", [0, 31], 1024, [(0, 0), (3, 517), (9, 1023), (15, 64)]),
    # the last 2048 tokens of the 32768-token prompts; rank 256
    ("cfg3_8b_long", [0], 2048, [(1, 0), (2, 1031), (3, 2047)]),
])
def test_prefill_chunk_at_full_size(name, layer_ids, T, picks):
    """lorc_prefill_attn on the benchmark's shapes: the last T tokens of every prompt attend to the whole cached
    prompt; sampled (sequence, query) rows against the oracle's decode attention over the cache rows the device holds,
    cut after the query's own token."""
    import torch
    sys.path.insert(0, ROOT)
    import bench
    from workloads import device as wdev
    L = helpers.lib()
    shape = synth.CONFIGS[name]
    device = torch.device("cuda", 0)
    wl = bench.Workload(L, shape, len(layer_ids), 1, device, 0, layer_ids=layer_ids, seeded_cache=True)
    N = shape.context
    ws = torch.zeros(L.lorc_prefill_workspace_bytes(wl.ctx, shape.batch, wl.n_max, T), dtype=torch.uint8, device=device)
    L.lorc_set_workspace(wl.ctx, ws)
    worst = 0.0
    for l, lid in enumerate(layer_ids):
        r = shape.ranks[lid]
        fac = _factors(shape, lid, r, device)
        q = wdev.queries((shape.batch, T, shape.n_q_heads, shape.d_head), lid, 555, device, 8.0)
        out = torch.zeros(shape.batch, T, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
        L.lorc_prefill_attn(wl.ctx, l, wl.caches[l], q, out, T)
        torch.cuda.synchronize()
        assert L.lorc_sync_status(wl.ctx) == 0, L.lorc_last_error(wl.ctx)
        assert L.lorc_last_path(wl.ctx) == 2
        for (s, t) in picks:
            n_t = N - T + t + 1
            ck, cv = _f64(wl.keep[l][0][s, :n_t]), _f64(wl.keep[l][1][s, :n_t])
            want = O.decode_attn_latent(ck, cv, fac["k"][1], fac["v"][1], _f64(q[s, t]), shape.n_kv_heads, shape.rope_theta)
            got = _f64(out[s, t])
            helpers.assert_rows_close(got, want, TOL, (name, lid, s, t), elem_factor=4.0)
            worst = max(worst, O.rel_l2_rows(got, want))
    print(f"\n[full size] prefill chunk of {T} on {name}, layers {layer_ids}: max relative L2 row error {worst:.2e}")
    wl.close()
    del ws
    torch.cuda.empty_cache()
