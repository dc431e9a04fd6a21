"""Context-sharded decode on one GPU: the shards of a context are attended to one after the other (the calls that R
ranks would make), then merged; every shard result and the merged result are compared with the fp64 oracle, and the
merged result with the unsharded call.  Both the tensor-core path and the plain kernels."""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _shard_caches(sess, lens, pos0, cnt, ck, cv, n_max):
    held = []
    for r in range(len(pos0)):
        kr = [ck[s][pos0[r][s]:pos0[r][s] + cnt[r][s]] for s in range(len(lens))]
        vr = [cv[s][pos0[r][s]:pos0[r][s] + cnt[r][s]] for s in range(len(lens))]
        held.append(H.contiguous_cache(sess, len(lens), n_max, cnt[r], kr, vr))
    return held


@pytest.mark.parametrize("geom,flags,path", [
    (dict(D=1024, H_q=32, H_kv=8, d_h=128, r_k=160, r_v=96), 0, 2),       # tcgen05 kernels
    (dict(D=256, H_q=8, H_kv=2, d_h=64, r_k=40, r_v=24), 1, 1),           # plain kernels, fp32 debug flag
])
@pytest.mark.parametrize("world", [2, 3])
def test_sharded_decode_equals_unsharded_and_oracle(geom, flags, path, world):
    import torch
    from paper_2410_03111_b200 import sharded
    L = H.lib()
    lens = [700, 130, 300, 17]           # the last two leave ranks with few or no rows
    prob = H.Problem(geom["D"], geom["H_q"], geom["H_kv"], geom["d_h"], geom["r_k"], geom["r_v"], theta=500000.0, layer=7)
    b, n_max = len(lens), 768
    sess = H.Session(prob, max_pos=n_max, batch=b, flags=flags)
    xs = [synth.hidden_states(n, prob.D, 7, chunk=50 + s).astype(np.float64) for s, n in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    q = synth.queries(b, prob.H_q, prob.d_h, 7, 2, 8.0).astype(np.float64)
    qd = H.dev_bf16(q)
    pos0, cnt = sharded.shard_bounds(lens, world)
    held = _shard_caches(sess, lens, pos0, cnt, ck, cv, n_max)
    q_pos = torch.tensor([n - 1 for n in lens], dtype=torch.int32, device="cuda")
    outs = torch.zeros(world, b, prob.H_q, prob.d_h, dtype=torch.bfloat16, device="cuda")
    mls = torch.zeros(world, b, prob.H_q, 2, dtype=torch.float32, device="cuda")
    for r in range(world):
        p0 = torch.tensor(pos0[r], dtype=torch.int32, device="cuda")
        L.lorc_decode_attn_shard(sess.ctx, 0, held[r][0], qd, p0, q_pos, outs[r], mls[r])
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == path
        ml = H.host_f64(mls[r])
        for s in range(b):
            a, n = pos0[r][s], cnt[r][s]
            if n == 0:
                assert np.all(ml[s, :, 1] == 0.0) and np.all(H.host_f64(outs[r, s]) == 0.0)
                continue
            pos = np.arange(a, a + n)
            want_lse = O.shard_log2_sum_exp(ck[s][a:a + n], prob.B_k, q[s], prob.H_kv, prob.theta, pos, lens[s] - 1)
            got_lse = ml[s, :, 0] + np.log2(ml[s, :, 1])
            assert np.max(np.abs(got_lse - want_lse)) <= 2e-2         # log2 units: 1.4 % of the shard's weight
            want_o = O.decode_attn_latent(ck[s][a:a + n], cv[s][a:a + n], prob.B_k, prob.B_v, q[s], prob.H_kv, prob.theta,
                                          positions=pos, q_position=lens[s] - 1)
            assert O.rel_l2_rows(H.host_f64(outs[r, s]), want_o) <= TOL
    merged = torch.zeros(b, prob.H_q, prob.d_h, dtype=torch.bfloat16, device="cuda")
    L.lorc_merge_shards(sess.ctx, world, outs, mls, merged, b)
    assert L.lorc_sync_status(sess.ctx) == 0
    want = H.oracle_decode(prob, ck, cv, q)
    # two bf16 roundings (shard outputs, merged output) instead of one
    H.assert_rows_close(H.host_f64(merged), want, 1.5 * TOL, ("merged", world))
    whole = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    ref = torch.zeros_like(merged)
    L.lorc_decode_attn(sess.ctx, 0, whole[0], qd, ref)
    assert L.lorc_sync_status(sess.ctx) == 0
    assert O.rel_l2_rows(H.host_f64(merged), H.host_f64(ref)) <= 1.5 * TOL
    sess.close()


def test_shard_rejects_query_before_the_shard_end_and_full_layers():
    import torch
    L = H.lib()
    prob = H.Problem(256, 8, 2, 64, 40, 24, layer=8)
    sess = H.Session(prob, max_pos=256, batch=1, flags=1)
    held = H.contiguous_cache(sess, 1, 256, [100])
    q = torch.zeros(1, 8, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 8, 64, dtype=torch.bfloat16, device="cuda")
    ml = torch.zeros(1, 8, 2, dtype=torch.float32, device="cuda")
    p0 = torch.tensor([50], dtype=torch.int32, device="cuda")
    for bad in (148, 256):             # before the shard's last token (149); beyond the rotation table
        L.lorc_decode_attn_shard(sess.ctx, 0, held[0], q, p0, torch.tensor([bad], dtype=torch.int32, device="cuda"), out, ml)
        assert L.lorc_sync_status(sess.ctx) == L.LORC_ERR_CAPACITY
    L.lorc_decode_attn_shard(sess.ctx, 0, held[0], q, p0, torch.tensor([149], dtype=torch.int32, device="cuda"), out, ml)
    assert L.lorc_sync_status(sess.ctx) == 0
    with pytest.raises(L.LorcError) as e:
        L.lorc_merge_shards(sess.ctx, 65, out, ml, out, 1)
    assert e.value.code == L.LORC_ERR_ARG
    sess.close()
    full = H.Session(prob, max_pos=256, batch=1, flags=1, mode=1)
    held = H.contiguous_cache(full, 1, 256, [100])
    with pytest.raises(L.LorcError) as e:
        L.lorc_decode_attn_shard(full.ctx, 0, held[0], q, p0, p0, out, ml)
    assert e.value.code == L.LORC_ERR_UNSUPPORTED
    full.close()
