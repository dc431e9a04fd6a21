"""Shared set-up for the GPU parity tests: inputs come from `workloads`, expected
values from `oracle`; the CUDA path is reached only through the C-ABI binding."""
from __future__ import annotations

import numpy as np

from oracle import lorc_oracle as O
from workloads import synth


ROPE_NONE = 2          # LORC_ROPE_NONE: no rotation at attention time


def lib():
    import paper_2410_03111_b200 as pkg
    return pkg.load()


def dev_bf16(a):
    """Upload bf16-exact float values as a torch bf16 CUDA tensor."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).cuda()


def host_f64(t):
    """Download a torch tensor as fp64 numpy."""
    return t.detach().float().cpu().numpy().astype(np.float64)


class Problem:
    """One layer's factors (bf16-exact) plus geometry."""

    def __init__(self, D, H_q, H_kv, d_h, r_k, r_v, theta=10000.0, p=0.8, layer=0, style=0):
        self.D, self.H_q, self.H_kv, self.d_h = D, H_q, H_kv, d_h
        self.n = H_kv * d_h
        self.r_k, self.r_v, self.theta, self.style, self.layer = r_k, r_v, theta, style, layer
        Uk, sk, Vk = synth.synth_weight_factors(D, self.n, p, layer, "k")
        Uv, sv, Vv = synth.synth_weight_factors(D, self.n, p, layer, "v")
        Ak, Bk = O.factors_from_generators(Uk, sk, Vk, r_k)
        Av, Bv = O.factors_from_generators(Uv, sv, Vv, r_v)
        # the factors the device holds are bf16; the oracle sees the same rounded values
        self.A_k, self.B_k = synth.to_bf16_exact(Ak), synth.to_bf16_exact(Bk)
        self.A_v, self.B_v = synth.to_bf16_exact(Av), synth.to_bf16_exact(Bv)
        self.W_k = synth.to_bf16_exact((Uk * sk) @ Vk.T)
        self.W_v = synth.to_bf16_exact((Uv * sv) @ Vv.T)


class Session:
    """A library context with one or more layers loaded, and a workspace."""

    def __init__(self, prob, max_pos, batch, flags=0, mode=0, n_layers=1):
        import torch
        self.L = lib()
        self.prob = prob
        self.ctx = self.L.lorc_create(n_layers, prob.D, prob.H_q, prob.H_kv, prob.d_h, prob.theta,
                                      rope_style=prob.style, max_pos=max_pos, flags=flags)
        self.mode = mode
        if mode == self.L.LORC_MODE_LATENT:
            self.dev = [dev_bf16(a) for a in (prob.A_k, prob.B_k, prob.A_v, prob.B_v)]
            self.L.lorc_load_factors(self.ctx, 0, mode, prob.r_k, prob.r_v, *self.dev)
        else:
            wk, wv = dev_bf16(prob.W_k), dev_bf16(prob.W_v)
            self.L.lorc_load_factors(self.ctx, 0, mode, 0, 0, wk, None, wv, None)
        nbytes = self.L.lorc_workspace_bytes(self.ctx, batch, max_pos)
        self.ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        self.L.lorc_set_workspace(self.ctx, self.ws)

    def widths(self):
        if self.mode == self.L.LORC_MODE_LATENT:
            return self.prob.r_k, self.prob.r_v
        return self.prob.n, self.prob.n

    def close(self):
        import torch
        torch.cuda.synchronize()
        self.L.lorc_destroy(self.ctx)
        self.ctx = None


def contiguous_cache(sess, batch, n_max, lens, k_rows=None, v_rows=None):
    """Zeroed contiguous cache [batch, n_max, w]; optional per-sequence rows to pre-load."""
    import torch
    wk, wv = sess.widths()
    k = torch.zeros(batch, n_max, wk, dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(batch, n_max, wv, dtype=torch.bfloat16, device="cuda")
    if k_rows is not None:
        for s in range(batch):
            k[s, :k_rows[s].shape[0]] = dev_bf16(k_rows[s])
            v[s, :v_rows[s].shape[0]] = dev_bf16(v_rows[s])
    sl = torch.tensor(np.asarray(lens, dtype=np.int32), device="cuda")
    cache = sess.L.make_cache(k, v, sl, batch, int(max(1, max(lens))), seq_stride=n_max)
    return cache, k, v, sl


def paged_cache(sess, batch, lens, page_size, order_seed, k_rows=None, v_rows=None, extra_pages=3):
    """Zeroed paged cache with a seeded random physical page order."""
    import torch
    wk, wv = sess.widths()
    max_pages = max(1, max((int(l) + page_size - 1) // page_size for l in lens))
    n_pages = batch * max_pages + extra_pages
    order = synth.page_order(n_pages, base_seed=order_seed)
    pt = order[:batch * max_pages].reshape(batch, max_pages).astype(np.int32)
    k = torch.zeros(n_pages, page_size, wk, dtype=torch.bfloat16, device="cuda")
    v = torch.zeros(n_pages, page_size, wv, dtype=torch.bfloat16, device="cuda")
    if k_rows is not None:
        for s in range(batch):
            L = k_rows[s].shape[0]
            kr, vr = dev_bf16(k_rows[s]), dev_bf16(v_rows[s])
            for pg in range((L + page_size - 1) // page_size):
                a, b = pg * page_size, min(L, (pg + 1) * page_size)
                k[int(pt[s, pg]), :b - a] = kr[a:b]
                v[int(pt[s, pg]), :b - a] = vr[a:b]
    sl = torch.tensor(np.asarray(lens, dtype=np.int32), device="cuda")
    ptd = torch.tensor(pt, device="cuda")
    cache = sess.L.make_cache(k, v, sl, batch, int(max(1, max(lens))), page_table=ptd,
                              page_size=page_size, max_pages_per_seq=max_pages, n_pages=n_pages)
    return cache, k, v, sl, ptd, pt


def oracle_latents(prob, xs):
    """bf16 latents the cache must hold for hidden states xs (list of [N_s, D])."""
    ck = [O.append_latent_bf16(x, prob.A_k) for x in xs]
    cv = [O.append_latent_bf16(x, prob.A_v) for x in xs]
    return ck, cv


def oracle_decode(prob, ck, cv, q):
    """fp64 decode attention per sequence from given latents; q [b, H_q, d_h]."""
    out = np.empty((len(ck), prob.H_q, prob.d_h))
    for s in range(len(ck)):
        if prob.style == ROPE_NONE:
            out[s] = O.decode_attn_latent(ck[s], cv[s], prob.B_k, prob.B_v, q[s], prob.H_kv, prob.theta, use_rope=False)
        else:
            out[s] = O.decode_attn_latent(ck[s], cv[s], prob.B_k, prob.B_v, q[s], prob.H_kv, prob.theta, prob.style)
    return out


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (fp64 array)."""
    _, ex = np.frexp(np.asarray(x, dtype=np.float64))
    return np.ldexp(1.0, np.maximum(ex - 1, -126) - 7)


def assert_rows_close(got, want, tol, tag=None, elem_factor=2.0):
    """Both bounds the parity tests use on an output [.., H_q, d_h]: the relative L2 error of every (sequence, head)
    row, and element by element |got - want| <= 2 tol * rms(row) + one bf16 ulp of the expected value.  (The output is
    rounded to bf16 once, which alone is up to half an ulp; the rest of the error is spread over the 64 or 128
    elements of a row with an rms of at most tol * rms(row), so 2 tol * rms(row) leaves a single element some five
    standard deviations at the measured error level of 3e-3.  Tests with a million elements and a higher error level
    pass a larger elem_factor.)"""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    err = O.rel_l2_rows(got, want)
    assert err <= tol, (tag, "relative L2 row error", err)
    rms = np.sqrt(np.mean(want ** 2, axis=-1, keepdims=True))
    excess = np.abs(got - want) - (elem_factor * tol * rms + bf16_ulp(want))
    assert np.all(excess <= 0.0), (tag, "element-wise bound exceeded by", float(excess.max()))
