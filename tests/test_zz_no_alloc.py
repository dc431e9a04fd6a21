"""The allocation-free decode-attention entry point (collected last on purpose).

lorc_decode_attn_static serves hosts that cannot allocate device memory when they
call the library (a server whose own pool owns the whole GPU, a plug-in without an
allocator): its scratch is a fixed array inside the library.  The test calls it
through the C ABI twice in a row, with different inputs, and checks each result
against lorc_decode_attn on the same inputs; it must also refuse a problem whose
partial results cannot fit the fixed array.
"""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    import torch
    D, H_q, H_kv, d_h, r_k, r_v = 512, 8, 2, 128, 96, 72
    lens = [700, 37, 300]
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=500000.0, layer=40)
    b = len(lens)
    # the plain kernels on both sides, so that the only difference is where the scratch lives
    sess = H.Session(prob, max_pos=768, batch=b, flags=sess_flags())
    xs = [synth.hidden_states(L, D, 40, chunk=s).astype(np.float64) for s, L in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    cache, k, v, sl = H.contiguous_cache(sess, b, 768, lens, ck, cv)
    for call, (q_scale, n_splits) in enumerate([(8.0, 0), (1.0, 3)]):
        q = synth.queries(b, H_q, d_h, 40, call, q_scale)
        ref = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        got = torch.full((b, H_q, d_h), 7.0, dtype=torch.bfloat16, device="cuda")
        sess.L.lorc_decode_attn(sess.ctx, 0, cache, H.dev_bf16(q), ref, n_splits=n_splits)
        sess.L.lorc_decode_attn_static(sess.ctx, 0, cache, H.dev_bf16(q), got, n_splits=n_splits)
        assert sess.L.lorc_sync_status(sess.ctx) == 0
        assert O.rel_l2_rows(H.host_f64(got), H.host_f64(ref)) <= 1e-2
        want = H.oracle_decode(prob, ck, cv, q.astype(np.float64))
        assert O.rel_l2_rows(H.host_f64(got), want) <= 1e-2
    # it works without any workspace lent to the context
    sess.L.lorc_set_workspace(sess.ctx, None)
    got2 = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn_static(sess.ctx, 0, cache, H.dev_bf16(q), got2, n_splits=3)
    assert sess.L.lorc_sync_status(sess.ctx) == 0
    assert torch.equal(got2, got)
    sess.close()


def sess_flags():
    return H.lib().LORC_FLAG_DEBUG_FP32


def test_static_scratch_entry_rejects_what_cannot_fit():
    import torch
    L = H.lib()
    D, H_q, H_kv, d_h, r = 256, 16, 2, 64, 128
    prob = H.Problem(D, H_q, H_kv, d_h, r, r, layer=41)
    b = 1100            # 1100 * 16 heads * (2 + 128) * 4 B > 8 MiB even with one split
    sess = H.Session(prob, max_pos=32, batch=b, flags=L.LORC_FLAG_DEBUG_FP32)
    k = torch.zeros(b, 32, r, dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(b, 32, r, dtype=torch.bfloat16, device="cuda")
    sl = torch.full((b,), 4, dtype=torch.int32, device="cuda")
    cache = L.make_cache(k, v, sl, b, 32, seq_stride=32)
    q = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    assert b * H_q * (2 + r) * 4 > L.LORC_STATIC_SCRATCH_BYTES
    with pytest.raises(L.LorcError) as e:
        L.lorc_decode_attn_static(sess.ctx, 0, cache, q, out)
    assert e.value.code == L.LORC_ERR_WORKSPACE
    assert "LORC_STATIC_SCRATCH_BYTES" in str(e.value)
    sess.close()
