"""The bounded device-side wait, made to run out on purpose in the one harmless way: a one-thread kernel waits, with the
routine every kernel of the library waits with, for 20 ms on a barrier that nothing signals.  It must come back with
status TIMEOUT (no trap, no hang), and the context must work afterwards."""
import time

import numpy as np
import pytest

from oracle import lorc_oracle as O
from workloads import synth

import helpers as H

pytestmark = pytest.mark.gpu


def test_wait_expiry_reports_timeout_and_context_stays_usable():
    import torch
    L = H.lib()
    prob = H.Problem(256, 8, 2, 64, 40, 24, layer=30)
    lens = [130, 47]
    sess = H.Session(prob, max_pos=160, batch=2)
    xs = [synth.hidden_states(n, prob.D, 30, chunk=s).astype(np.float64) for s, n in enumerate(lens)]
    ck, cv = H.oracle_latents(prob, xs)
    held = H.contiguous_cache(sess, 2, 160, lens, ck, cv)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    L.lorc_selftest_wait_expiry(sess.ctx, 20_000_000)
    assert L.lorc_sync_status(sess.ctx) == L.LORC_ERR_TIMEOUT
    dt = time.perf_counter() - t0
    assert 0.015 <= dt <= 1.0, dt                     # it waited for its limit, and not for the library's 2 s
    assert L.lorc_sync_status(sess.ctx) == 0          # reading the status cleared it
    # the limit is bounded on the host side too
    with pytest.raises(L.LorcError) as e:
        L.lorc_selftest_wait_expiry(sess.ctx, 5_000_000_000)
    assert e.value.code == L.LORC_ERR_ARG
    # the context still works
    q = synth.queries(2, prob.H_q, prob.d_h, 30, 1, 8.0).astype(np.float64)
    out = torch.zeros(2, prob.H_q, prob.d_h, dtype=torch.bfloat16, device="cuda")
    L.lorc_decode_attn(sess.ctx, 0, held[0], H.dev_bf16(q), out)
    assert L.lorc_sync_status(sess.ctx) == 0
    assert O.rel_l2_rows(H.host_f64(out), H.oracle_decode(prob, ck, cv, q)) <= 1e-2
    sess.close()
