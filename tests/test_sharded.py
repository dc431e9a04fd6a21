"""Context-sharded decode: the oracle's merge pinned to attention over the whole context, the split planner, and the
exchange run on two gloo ranks with the oracle standing in for the two kernels."""
import math
import os
import socket
import sys

import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _problem(N=50, D=32, H_q=4, H_kv=2, d=8, r_k=12, r_v=10, seed=3):
    rng = np.random.default_rng(seed)
    ck = rng.standard_normal((N, r_k))
    cv = rng.standard_normal((N, r_v))
    B_k = rng.standard_normal((r_k, H_kv * d))
    B_v = rng.standard_normal((r_v, H_kv * d))
    q = 3.0 * rng.standard_normal((H_q, d))
    return ck, cv, B_k, B_v, q, H_kv


@pytest.mark.parametrize("cuts", [[0, 20, 50], [0, 1, 2, 50], [0, 50, 50], [0, 0, 17, 50]])
def test_merge_of_shards_is_attention_over_the_whole_context(cuts):
    ck, cv, B_k, B_v, q, H_kv = _problem()
    N, theta = ck.shape[0], 10000.0
    whole = O.decode_attn_latent(ck, cv, B_k, B_v, q, H_kv, theta)
    outs, sums = [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        pos = np.arange(a, b)
        sums.append(O.shard_log2_sum_exp(ck[a:b], B_k, q, H_kv, theta, pos, N - 1))
        outs.append(O.decode_attn_latent(ck[a:b], cv[a:b], B_k, B_v, q, H_kv, theta, positions=pos, q_position=N - 1)
                    if b > a else np.zeros_like(whole))
    got = O.merge_context_shards(np.stack(outs), np.stack(sums))
    assert np.max(np.abs(got - whole)) <= 1e-12 * np.max(np.abs(whole))


def test_log2_sum_exp_against_brute_force_and_closed_forms():
    ck, cv, B_k, B_v, q, H_kv = _problem(N=7)
    theta = 10000.0
    got = O.shard_log2_sum_exp(ck, B_k, q, H_kv, theta, np.arange(7), 6)
    # brute force, scalar loops: rotate by hand with the closed form of the rotation of pair (j, j + d/2)
    H_q, d = q.shape
    G = H_q // H_kv

    def rot(v, p):
        w = np.array(v, dtype=float)
        for j in range(d // 2):
            ang = p * theta ** (-2.0 * j / d)
            w[j] = v[j] * math.cos(ang) - v[j + d // 2] * math.sin(ang)
            w[j + d // 2] = v[j] * math.sin(ang) + v[j + d // 2] * math.cos(ang)
        return w

    for h in range(H_q):
        tot = 0.0
        for n in range(7):
            k = (ck[n] @ B_k)[(h // G) * d:(h // G + 1) * d]
            tot += math.exp(float(rot(k, n) @ rot(q[h], 6)) / math.sqrt(d))
        assert got[h] == pytest.approx(math.log2(tot), rel=1e-12, abs=1e-12)
    # zero query: every score is 0, the sum is N; no rows: -inf
    zero = O.shard_log2_sum_exp(ck, B_k, np.zeros_like(q), H_kv, theta, np.arange(7), 6)
    assert np.allclose(zero, math.log2(7), rtol=0, atol=1e-14)
    assert np.all(np.isneginf(O.shard_log2_sum_exp(ck[:0], B_k, q, H_kv, theta, np.arange(0), 6)))


def test_merge_closed_forms():
    a, b = np.array([[1.0, 2.0]]), np.array([[3.0, 6.0]])
    # equal weights: the mean; a shard one unit higher in log2 counts twice; an empty shard drops out
    assert np.allclose(O.merge_context_shards(np.stack([a, b]), np.array([[0.5], [0.5]])), [[2.0, 4.0]])
    assert np.allclose(O.merge_context_shards(np.stack([a, b]), np.array([[0.0], [1.0]])), [[7.0 / 3, 14.0 / 3]])
    assert np.allclose(O.merge_context_shards(np.stack([a, b]), np.array([[-np.inf], [-3.0]])), b)
    # very different magnitudes neither overflow nor lose the dominant shard
    assert np.allclose(O.merge_context_shards(np.stack([a, b]), np.array([[4000.0], [-4000.0]])), a)


def test_shard_bounds_cover_every_position_once():
    from paper_2410_03111_b200 import sharded
    lens = [0, 1, 127, 128, 129, 1000, 32768]
    for world in (1, 2, 3, 8):
        pos0, cnt = sharded.shard_bounds(lens, world)
        for s, n in enumerate(lens):
            at = 0
            for r in range(world):
                assert pos0[r][s] == at and cnt[r][s] >= 0
                assert pos0[r][s] % 128 == 0 or cnt[r][s] == 0
                at += cnt[r][s]
            assert at == n
            full = [cnt[r][s] for r in range(world)]
            assert max(full) - min(full) <= 128 + 127
    assert sharded.append_owner([0, 127, 128, 255, 256], 2) == [0, 0, 1, 1, 1]
    assert sharded.append_owner([383, 384], 2) == [1, 1]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out_q):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2410_03111_b200 import sharded
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ck, cv, B_k, B_v, q, H_kv = _problem(N=300, d=8)
    lens, theta = [300, 140], 10000.0
    H_q, d = q.shape
    qs = np.stack([q, -0.5 * q])
    pos0, cnt = sharded.shard_bounds(lens, world)

    # stand-ins with the library calls' signatures: the oracle on this rank's rows
    def attend(ctx, layer, cache, q_t, p0_t, qp_t, o_t, ml_t, n_splits, stream):
        for s in range(len(lens)):
            a, n = int(p0_t[s]), cache[s]
            pos = np.arange(a, a + n)
            lse = O.shard_log2_sum_exp(ck[a:a + n], B_k, qs[s], H_kv, theta, pos, int(qp_t[s]))
            o = (O.decode_attn_latent(ck[a:a + n], cv[a:a + n], B_k, B_v, qs[s], H_kv, theta, positions=pos,
                                      q_position=int(qp_t[s])) if n else np.zeros((H_q, d)))
            o_t[s] = torch.from_numpy(o).to(torch.bfloat16)
            # any split of the sum into a reference and a remainder is valid: use a different one on each rank
            ref = np.where(np.isfinite(lse), np.ceil(lse) + rank, 0.0)
            ml_t[s, :, 0] = torch.from_numpy(ref).float()
            ml_t[s, :, 1] = torch.from_numpy(np.where(np.isfinite(lse), np.exp2(lse - ref), 0.0)).float()

    def merge(ctx, n_shards, outs, mls, out, batch, stream):
        assert n_shards == world and tuple(outs.shape) == (world, batch, H_q, d)
        lse = np.where(mls[..., 1].numpy() > 0, mls[..., 0].double().numpy() + np.log2(np.maximum(mls[..., 1].double().numpy(), 1e-300)), -np.inf)
        out.copy_(torch.from_numpy(O.merge_context_shards(outs.double().numpy(), lse)).to(torch.bfloat16))

    dec = sharded.ShardedDecoder(None, H_q, d, group=None, attend=attend, merge=merge)
    out = torch.zeros(len(lens), H_q, d, dtype=torch.bfloat16)
    dec.decode(0, cnt[rank], torch.zeros(len(lens), H_q, d), torch.tensor(pos0[rank], dtype=torch.int32),
               torch.tensor([n - 1 for n in lens], dtype=torch.int32), out)
    dist.barrier()
    out_q.put((rank, out.double().numpy()))
    dist.destroy_process_group()


def test_sharded_decode_two_gloo_ranks():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out_q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out_q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    ck, cv, B_k, B_v, q, H_kv = _problem(N=300, d=8)
    want = np.stack([O.decode_attn_latent(ck[:300], cv[:300], B_k, B_v, q, H_kv, 10000.0),
                     O.decode_attn_latent(ck[:140], cv[:140], B_k, B_v, -0.5 * q, H_kv, 10000.0)])
    assert np.array_equal(res[0], res[1])                    # every rank ends with the same result
    assert O.rel_l2_rows(res[0], want) <= 1.5e-2             # two bf16 roundings (shard outputs, merged output)
