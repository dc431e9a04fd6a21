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


@pytest.mark.parametrize("variant", ["full_layer", "paged_bf16_path", "splits_lowered_to_fit"])
def test_static_scratch_entry_other_shapes(variant):
    """The same comparison for an uncompressed layer with 128-wide heads (the streaming kernel fills the fixed array),
    for a paged cache on a context without the debug flag, and for a batch whose partial results only fit after the
    split count has been lowered."""
    import torch
    L = H.lib()
    if variant == "full_layer":
        D, H_q, H_kv, d_h, r_k, r_v, lens, flags, mode = 256, 8, 2, 128, 256, 256, [150, 33], 0, 1
    elif variant == "paged_bf16_path":
        D, H_q, H_kv, d_h, r_k, r_v, lens, flags, mode = 256, 8, 2, 64, 40, 24, [130, 47, 64], 0, 0
    else:
        # 94 splits are asked for (one per 32-token tile): 56 sequences x 8 heads x 94 x (2 + 64) x 4 B = 11.1 MiB do not
        # fit the 8 MiB array, so the entry point lowers the split count until they do
        D, H_q, H_kv, d_h, r_k, r_v, lens, flags, mode = 128, 8, 2, 64, 16, 64, [3000] * 56, 1, 0
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=10000.0, layer=42)
    b, n_max = len(lens), max(lens) + 8
    sess = H.Session(prob, max_pos=n_max, batch=b, flags=flags, mode=mode)
    if mode == 1:
        held = H.contiguous_cache(sess, b, n_max, [max(lens)] * b)
        x = np.stack([synth.hidden_states(max(lens), D, 42, chunk=s) for s in range(b)]).astype(np.float64)
        L.lorc_append(sess.ctx, 0, held[0], H.dev_bf16(x), T=max(lens))
        held[3][:] = torch.tensor(lens, dtype=torch.int32)
    else:
        if len(set(lens)) == 1:
            one = H.oracle_latents(prob, [synth.hidden_states(lens[0], D, 42).astype(np.float64)])
            ck, cv = [one[0][0]] * b, [one[1][0]] * b
        else:
            ck, cv = H.oracle_latents(prob, [synth.hidden_states(n, D, 42, chunk=s).astype(np.float64) for s, n in enumerate(lens)])
        if variant == "paged_bf16_path":
            held = H.paged_cache(sess, b, lens, 16, order_seed=3, k_rows=ck, v_rows=cv)
        else:
            held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    q = H.dev_bf16(synth.queries(b, H_q, d_h, 42, 1, 8.0))
    n_splits = 94 if variant == "splits_lowered_to_fit" else 0
    if n_splits:
        assert b * H_q * n_splits * (2 + r_v) * 4 > L.LORC_STATIC_SCRATCH_BYTES
    for call in range(2):
        ref = torch.zeros(b, H_q, d_h, dtype=torch.bfloat16, device="cuda")
        got = torch.full((b, H_q, d_h), 3.0, dtype=torch.bfloat16, device="cuda")
        L.lorc_decode_attn(sess.ctx, 0, held[0], q, ref, n_splits=n_splits)
        path_ref = L.lorc_last_path(sess.ctx)
        L.lorc_decode_attn_static(sess.ctx, 0, held[0], q, got, n_splits=n_splits)
        assert L.lorc_sync_status(sess.ctx) == 0, L.lorc_last_error(sess.ctx)
        assert L.lorc_last_path(sess.ctx) == path_ref == (3 if variant == "full_layer" else 1)
        assert O.rel_l2_rows(H.host_f64(got), H.host_f64(ref)) <= 1e-2
    sess.close()
