"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The workload object of bench.py is built for a whole configuration (all sequences, the full context, the
library's own prefill), one decode step is launched call by call and a second one as a CUDA-graph replay, exactly
as the benchmark does.  The oracle cannot redo all of that, so it redoes sampled (layer, sequence) outputs one by
one, from the seeded inputs alone: it derives the factors from the weight generators, the latents from the hidden
states (Sec. 3.1) and the attention output from those (Sec. 3.3 with the position embedding applied at attention
time).  Nothing the CUDA path produced enters the oracle.
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

CASES = [
    # configuration, layers built, sampled (layer, sequence) pairs
    ("cfg2_8b_progressive", 32, [(0, 3), (13, 0), (31, 15)]),
    ("cfg3_8b_long", 1, [(0, 2)]),
    ("cfg4_70b_progressive", 2, [(1, 5)]),
]


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


@pytest.mark.gpu
@pytest.mark.parametrize("name,n_layers,samples", CASES, ids=[c[0] for c in CASES])
def test_sampled_outputs_at_full_size(name, n_layers, samples):
    import torch
    sys.path.insert(0, ROOT)
    import bench
    from workloads import device as wdev
    L = helpers.lib()
    shape = synth.CONFIGS[name]
    device = torch.device("cuda", 0)
    wl = bench.Workload(L, shape, n_layers, 4, device, 0)
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
    chunk = 512
    for (l, s) in samples:
        r = shape.ranks[l]
        # factors from the generators of the synthetic weights, rounded to bf16 as the library holds them
        fac = {}
        for which in ("k", "v"):
            U, sg, V = wdev.weight_generators(shape.d_model, shape.n, shape.sigma_p, l, which, device)
            A, B = O.factors_from_generators(_f64(U), _f64(sg), _f64(V), r)
            fac[which] = (synth.to_bf16_exact(A), synth.to_bf16_exact(B))
            del U, V
        # hidden states of this sequence: the prefill chunks, then the decode steps
        xs = [_f64(wdev.hidden_states((shape.batch, min(chunk, shape.context - c0), shape.d_model), l, c0 // chunk,
                                      device)[s]) for c0 in range(0, shape.context, chunk)]
        xs += [_f64(wl.x[l][i][s])[None, :] for i in range(steps_done)]
        X = np.concatenate(xs, axis=0)
        assert X.shape == (N, shape.d_model)
        ck = O.append_latent_bf16(X, fac["k"][0])
        cv = O.append_latent_bf16(X, fac["v"][0])
        # cache write: the device's latents against the exactly rounded ones
        # Bound: one bf16 ulp of the exact latent (the final rounding may fall either way) plus the fp32 accumulation
        # error of a D-term dot product, taken as 2^-16 of sum_i |x_i A_ij| (between the typical sqrt(D) 2^-24 and the
        # worst case D 2^-24 for D = 4096 ... 8192); the second term only matters where the terms cancel to a latent
        # far smaller than themselves.
        for ref, dev, A in ((ck, wl.keep[l][0], fac["k"][0]), (cv, wl.keep[l][1], fac["v"][0])):
            got = _f64(dev[s, :N])
            err = np.abs(got - ref)
            bound = helpers.bf16_ulp(ref) + 2.0 ** -16 * (np.abs(X) @ np.abs(A))
            assert np.all(err <= bound), float((err / bound).max())
            assert np.mean(err > 0) < 0.02          # a different last bit only where fp32 and fp64 sums straddle a tie
        q = _f64(wl.q[l][steps_done - 1][s])
        want = O.decode_attn_latent(ck, cv, fac["k"][1], fac["v"][1], q, shape.n_kv_heads, shape.rope_theta)
        got = _f64(wl.out[l, s])
        assert np.all(np.isfinite(got))
        assert O.rel_l2_rows(got, want) <= TOL, (name, l, s, O.rel_l2_rows(got, want))
    del wl
    torch.cuda.empty_cache()


RAGGED = ["cfg5_ragged_r384", "cfg5_ragged_r1024"]


@pytest.mark.gpu
@pytest.mark.parametrize("name", RAGGED)
def test_ragged_paged_batch_at_full_size(name):
    """64 sequences of 512 ... 16384 tokens in 64-token pages scattered over the pool: the shortest, the longest and
    two more sequences against the oracle, which reads the same seeded cache rows through the same page table."""
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
    q = wdev.queries((shape.batch, shape.n_q_heads, shape.d_head), 0, 0, device, 8.0)
    out = torch.zeros(shape.batch, shape.n_q_heads, shape.d_head, dtype=torch.bfloat16, device=device)
    L.lorc_decode_attn(sess.ctx, 0, cache, q, out)
    torch.cuda.synchronize()
    assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
    assert L.lorc_last_path(sess.ctx) == 2
    got_all = _f64(out)
    assert np.all(np.isfinite(got_all))
    order = np.argsort(lens)
    picks = [int(order[0]), int(order[-1]), int(order[len(order) // 3]), int(order[2 * len(order) // 3])]
    ps = shape.page_size
    for s in picks:
        n = int(lens[s])
        pages = torch.tensor(pt[s, :(n + ps - 1) // ps].astype(np.int64), device=device)
        ck = _f64(k[pages].reshape(-1, r)[:n])
        cv = _f64(v[pages].reshape(-1, r)[:n])
        want = O.decode_attn_latent(ck, cv, prob.B_k, prob.B_v, _f64(q[s]), shape.n_kv_heads, shape.rope_theta)
        err = O.rel_l2_rows(got_all[s], want)
        assert err <= TOL, (name, s, n, err)
    sess.close()
    del k, v
    torch.cuda.empty_cache()
