"""GPU parity of prompt processing (lorc_prefill_attn) against the fp64 oracle, through the C ABI.

The T newest tokens of every sequence attend to the cached prefix in full and to their own chunk causally.  Cases on
the plain kernels (small heads, fp32 debug path and bf16 path) and on the tensor-core path (8B head geometry:
reconstruction of keys and values on tcgen05, then a flash-attention kernel), contiguous and paged caches, chunks that
do not fill the last query block, a chunk that is the whole sequence, and T = 1 against decode attention.
"""
import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _oracle_prefill(prob, ck, cv, q, T):
    out = np.empty(q.shape)
    for s in range(len(ck)):
        out[s] = O.prefill_attn_latent(ck[s], cv[s], prob.B_k, prob.B_v, q[s], prob.H_kv, prob.theta,
                                       use_rope=prob.style != H.ROPE_NONE)
    return out


def _run_prefill(sess, cache, q, T, b, H_q, d_h, batch_ws):
    import torch
    need = sess.L.lorc_prefill_workspace_bytes(sess.ctx, b, batch_ws, T)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    sess.L.lorc_set_workspace(sess.ctx, ws)
    out = torch.zeros(b, T, H_q, d_h, dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_prefill_attn(sess.ctx, 0, cache, H.dev_bf16(q), out, T)
    assert sess.L.lorc_sync_status(sess.ctx) == 0, sess.L.lorc_last_error(sess.ctx)
    return out, ws


@pytest.mark.parametrize("flags", [1, 0])
def test_prefill_plain_kernels(flags):
    D, H_q, H_kv, d_h, r_k, r_v = 256, 4, 2, 64, 40, 24
    lens, T = [150, 33], 7
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=10000.0, layer=12)
    sess = H.Session(prob, max_pos=160, batch=2, flags=flags)
    xs = [synth.hidden_states(L, D, 12, chunk=s).astype(np.float64) for s, L in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    held = H.contiguous_cache(sess, 2, 160, lens, ck, cv)
    q = synth.gaussian((2, T, H_q, d_h), 12, 77).astype(np.float32)
    q = synth.to_bf16_exact(4.0 * q).astype(np.float64)
    out, ws = _run_prefill(sess, held[0], q, T, 2, H_q, d_h, 160)
    assert sess.L.lorc_last_path(sess.ctx) == 1
    want = _oracle_prefill(prob, ck, cv, q, T)
    got = H.host_f64(out)
    assert O.rel_l2_rows(got, want) <= (1e-2 if not flags else 5e-3)
    sess.close()


GEOM = dict(D=1024, H_q=32, H_kv=8, d_h=128)


@pytest.mark.parametrize("r_k,r_v,lens,T,paged,style", [
    (96, 72, [300, 700], 130, False, 0),          # chunk after a prefix; 130 = 4 query blocks + 2 positions
    (256, 256, [129, 128, 1000], 128, True, 0),   # paged; for the 128-token sequence the chunk is the whole sequence
    (416, 416, [513], 513, False, 0),             # a whole prompt in one call
    (160, 160, [400, 90], 64, False, H.ROPE_NONE),
])
def test_prefill_tensor_core_path(r_k, r_v, lens, T, paged, style):
    prob = H.Problem(GEOM["D"], GEOM["H_q"], GEOM["H_kv"], GEOM["d_h"], r_k, r_v, theta=500000.0, layer=23, style=style)
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    xs = [synth.hidden_states(int(L), prob.D, 23, chunk=300 + s).astype(np.float64) for s, L in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    if paged:
        held = H.paged_cache(sess, b, lens, 64, order_seed=9, k_rows=ck, v_rows=cv)
    else:
        held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    worst = 0.0
    # (the keys are materialised in fp16: a score carries their rounding, 2^-11 of |q| |k|, which the most peaked
    # softmaxes here see)
    for scale in (1.0, 8.0, 64.0):
        q = synth.to_bf16_exact(scale * synth.gaussian((b, T, GEOM["H_q"], GEOM["d_h"]), 23, int(scale))).astype(np.float64)
        out, ws = _run_prefill(sess, held[0], q, T, b, GEOM["H_q"], GEOM["d_h"], max(lens))
        assert sess.L.lorc_last_path(sess.ctx) == 2, "the tensor-core path was not taken"
        got = H.host_f64(out)
        want = _oracle_prefill(prob, ck, cv, q, T)
        # (at scale 64 the error level is 6e-3 of a row and the outputs have up to two million elements: the
        # largest of so many needs the wider element bound)
        H.assert_rows_close(got, want, TOL, (r_k, T, scale), elem_factor=4.0 if scale > 8 else 2.0)
        worst = max(worst, O.rel_l2_rows(got, want))
    print(f"\n[prefill] r_k {r_k}, T {T}, lens {lens}: max relative L2 row error {worst:.2e}")
    sess.close()


def test_prefill_with_one_token_equals_decode():
    import torch
    prob = H.Problem(GEOM["D"], GEOM["H_q"], GEOM["H_kv"], GEOM["d_h"], 128, 128, theta=500000.0, layer=24)
    lens = [260, 77]
    sess = H.Session(prob, max_pos=300, batch=2)
    xs = [synth.hidden_states(int(L), prob.D, 24, chunk=s).astype(np.float64) for s, L in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    held = H.contiguous_cache(sess, 2, 300, lens, ck, cv)
    q = synth.queries(2, GEOM["H_q"], GEOM["d_h"], 24, 0, 8.0).astype(np.float64)
    dec = torch.zeros(2, GEOM["H_q"], GEOM["d_h"], dtype=torch.bfloat16, device="cuda")
    sess.L.lorc_decode_attn(sess.ctx, 0, held[0], H.dev_bf16(q), dec)
    out, ws = _run_prefill(sess, held[0], q[:, None], 1, 2, GEOM["H_q"], GEOM["d_h"], max(lens))
    want = H.oracle_decode(prob, ck, cv, q)
    assert O.rel_l2_rows(H.host_f64(out[:, 0]), want) <= TOL
    assert O.rel_l2_rows(H.host_f64(out[:, 0]), H.host_f64(dec)) <= TOL
    sess.close()


@pytest.mark.parametrize("lens,T", [([300, 150], 45), ([200], 200)])
def test_prefill_tensor_core_path_eight_heads_per_kv_head(lens, T):
    """The 70B head geometry (64 query heads, 8 per KV head): a block of 128 query rows is 16 positions, a CTA covers 32;
    T = 45 leaves the second block of the last CTA partly past the chunk."""
    D, H_q, H_kv, d_h, r_k, r_v = 1024, 64, 8, 128, 160, 96
    prob = H.Problem(D, H_q, H_kv, d_h, r_k, r_v, theta=500000.0, layer=25)
    b, n_max = len(lens), max(lens) + 3
    sess = H.Session(prob, max_pos=n_max, batch=b)
    xs = [synth.hidden_states(int(L), D, 25, chunk=400 + s).astype(np.float64) for s, L in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    held = H.contiguous_cache(sess, b, n_max, lens, ck, cv)
    for scale in (1.0, 8.0):
        q = synth.to_bf16_exact(scale * synth.gaussian((b, T, H_q, d_h), 25, int(scale))).astype(np.float64)
        out, ws = _run_prefill(sess, held[0], q, T, b, H_q, d_h, max(lens))
        assert sess.L.lorc_last_path(sess.ctx) == 2, "the tensor-core path was not taken"
        H.assert_rows_close(H.host_f64(out), _oracle_prefill(prob, ck, cv, q, T), TOL, (T, scale))
    sess.close()
