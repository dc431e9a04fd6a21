"""CPU oracle for LoRC latent-KV decode attention (arXiv 2410.03111).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy restatement of what
the paper's method computes on the decode path.  It exists to judge the CUDA
library and to be timed as a CPU baseline; the product never imports it, and it
imports nothing from the product.  No blocking, fusion or re-association beyond
what the paper states: keys and values are reconstructed explicitly from the
cached latents, rotated, and fed to the textbook attention formula.

Notation (row-vector convention, K = X W_k as in the Preliminary section):
  D        model dimension            n = H_kv * d_h   width of the concatenated KV heads
  W [D,n]  key or value weight        W ~= A B,  A = U_r Sigma_r [D,r],  B = V_r^T [r,n]
  C = X A  the latent ("compressed") cache row, width r = d_c        (Sec. 3.1)

Every function is pinned by tests/test_oracle_pins.py (the schedule functions by
tests/test_schedule.py, the context-shard functions by tests/test_sharded.py) to something the paper or
the mathematics fixes (full-rank identity, Eckart-Young, Theorem 1, RoPE closed
forms, brute-force attention, a library attention routine).  The numeric
tolerance used when comparing the GPU to this oracle is not from the paper
(parity tolerance unpinned by the paper; 1e-2 for bf16 operands with fp32 accumulation, 1e-5 for fp32 arithmetic).
"""
from __future__ import annotations

import math

import numpy as np

ROPE_HALF_SPLIT = 0    # pairs (j, j + d_h/2)
ROPE_INTERLEAVED = 1   # pairs (2j, 2j + 1)


# --------------------------------------------------------------------------
# rounding
# --------------------------------------------------------------------------
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 value (round to nearest, ties to even) of fp64 x, as fp64.

    bfloat16 keeps 8 significant bits over the float32 exponent range, so the
    spacing at |x| in [2^e, 2^(e+1)) is 2^(e-7), with e floored at -126
    (subnormals).  Rounding is done straight from fp64 (no float32 detour).
    The paper is silent on the cache precision; bf16 is the reading taken here.
    """
    x = np.asarray(x, dtype=np.float64)
    _, ex = np.frexp(x)                      # x = m * 2^ex, 0.5 <= |m| < 1
    e = np.maximum(ex - 1, -126)
    quantum = np.ldexp(1.0, e - 7)
    y = np.rint(x / quantum) * quantum       # np.rint rounds half to even
    big = 3.3895313892515355e38              # largest finite bf16
    y = np.where(np.abs(y) > big, np.copysign(np.inf, y), y)
    return np.where(x == 0.0, x, y)


# --------------------------------------------------------------------------
# factorisation (offline step; Sec. 3.1, Algorithm 1 "Key/Value Matrix Compression")
# --------------------------------------------------------------------------
def truncated_svd_factors(W: np.ndarray, r: int):
    """Rank-r factors of W [D,n]: A = U_r Sigma_r [D,r], B = V_r^T [r,n].

    Sec. 3.1 (the SVD equations for W_k^H and W_v^H) splits W into an
    orthonormal factor and a Sigma-carrying factor, and caches the product of X
    with the Sigma-carrying one.  In the row-vector convention K = X W used
    here, that cached quantity is X (U_r Sigma_r): Sigma stays on the cached
    side, the orthonormal factor V_r^T is applied at attention time.
    """
    U, s, Vt = np.linalg.svd(np.asarray(W, dtype=np.float64), full_matrices=False)
    return U[:, :r] * s[None, :r], Vt[:r, :].copy()


def factors_from_generators(U: np.ndarray, sigma: np.ndarray, V: np.ndarray, r: int):
    """Same factors when W = U diag(sigma) V^T is given by its SVD (sigma descending).

    Avoids the sign/rotation freedom of a numerical SVD: A = U[:, :r] diag(sigma[:r]),
    B = V[:, :r]^T.
    """
    return U[:, :r] * np.asarray(sigma, dtype=np.float64)[None, :r], V[:, :r].T.copy()


def relative_frobenius_error(M: np.ndarray, M_hat: np.ndarray) -> float:
    """epsilon = ||M - M_hat||_F / ||M||_F  (Appendix "Reconstruction Error of Matrix SVD")."""
    M = np.asarray(M, dtype=np.float64)
    d = M - np.asarray(M_hat, dtype=np.float64)
    return math.sqrt(float(np.sum(d * d))) / math.sqrt(float(np.sum(M * M)))


def kv_cache_elements(b: int, N: int, h: int, d: int) -> int:
    """Per-layer cache size C_{k,v} = b * N * h * d (Preliminary section, cache-size equation)."""
    return b * N * h * d


def compression_ratio(d_c: int, h: int, d: int) -> float:
    """rho = d_c / (h * d): the retained fraction of the cache width (Sec. 3.1, "Compression Ratio")."""
    return d_c / float(h * d)



# --------------------------------------------------------------------------
# progressive compression schedule (Sec. 3.2; Algorithm 1, the two loops before the matrix compression)
# --------------------------------------------------------------------------
def condition_number(W: np.ndarray) -> float:
    """kappa(W) = ||W||_2 ||W^+||_2 = sigma_max(W) / sigma_min(W)  (Sec. 3.2, the condition-number equation),
    sigma_min being the smallest of the min(D, n) singular values of W [D, n]."""
    s = np.linalg.svd(np.asarray(W, dtype=np.float64), compute_uv=False)
    return float(s[0] / s[-1])


def cumulative_log_condition(kappa_k, kappa_v) -> np.ndarray:
    """log of the cumulative condition numbers, log kappa~_l = sum_{j >= l} (log kappa(W_k^j) + log kappa(W_v^j))
    (Sec. 3.2, "Cumulative Condition Number": the product runs from layer l to the last layer).  Returned in log
    form because the product itself overflows for deep models; the compression-dimension equation only uses logs."""
    lk = np.log(np.asarray(kappa_k, dtype=np.float64)) + np.log(np.asarray(kappa_v, dtype=np.float64))
    L = lk.shape[0]
    out = np.empty(L, dtype=np.float64)
    acc = 0.0
    for l in range(L - 1, -1, -1):          # Algorithm 1 walks l = L .. 1
        acc += lk[l]
        out[l] = acc
    return out


def compression_dimensions(log_kappa_tilde, d_min: float, d_max: float) -> np.ndarray:
    """Real-valued d_c^l of the compression-dimension equation (Sec. 3.2, Eq. "dc"):
        d_c^l = d_max * [1 - (max_i log k~_i - log k~_l) / (max_i log k~_i - min_i log k~_i) * (1 - d_min / d_max)].
    The layer with the largest cumulative condition number keeps d_max, the one with the smallest d_min.
    When all layers are equally sensitive the fraction is 0/0; every layer then keeps d_max."""
    lk = np.asarray(log_kappa_tilde, dtype=np.float64)
    hi, lo = float(np.max(lk)), float(np.min(lk))
    if hi == lo:
        return np.full(lk.shape, float(d_max))
    return d_max * (1.0 - (hi - lk) / (hi - lo) * (1.0 - d_min / d_max))


def progressive_schedule(kappa_k, kappa_v, d_min: float, d_max: float, quantum: int = 1,
                         log_threshold=None):
    """Per-layer compression decision of Algorithm 1: (d_c [L] integers, skip [L] booleans).

    d_c is Eq. "dc" rounded to the nearest multiple of `quantum` (ties to even; at least one quantum): the paper's
    equation is real-valued and does not say how it is rounded (reading).  A layer is skipped
    ("Skip compression for layer l") when its cumulative condition number exceeds the threshold; the comparison is
    made on log kappa~_l against `log_threshold` because the product of 2 (L - l + 1) condition numbers is far
    beyond the thresholds the paper quotes (30, 90), whose scale it does not define (reading: a parameter)."""
    lk = cumulative_log_condition(kappa_k, kappa_v)
    d = compression_dimensions(lk, d_min, d_max)
    d = np.maximum(np.rint(d / quantum) * quantum, quantum).astype(np.int64)
    skip = np.zeros(lk.shape, dtype=bool) if log_threshold is None else lk > float(log_threshold)
    return d, skip

# --------------------------------------------------------------------------
# cache write (Sec. 3.1: the cache keeps X times the Sigma-carrying factor, for keys and for values)
# --------------------------------------------------------------------------
def append_latent(x: np.ndarray, A: np.ndarray) -> np.ndarray:
    """Exact latent rows C = X A, fp64, [n_tok, r].  No rotation is applied (Appendix
    "Adjusted Position Embedding": the cache holds un-rotated compressed keys)."""
    return np.asarray(x, dtype=np.float64) @ np.asarray(A, dtype=np.float64)


def append_latent_bf16(x: np.ndarray, A: np.ndarray) -> np.ndarray:
    """The value a bf16 cache must hold: the exact latent rounded once to bf16."""
    return bf16_round(append_latent(x, A))


# --------------------------------------------------------------------------
# rotary position embedding (Appendix "Adjusted Position Embedding", RoFormer's R_{Theta,p})
# --------------------------------------------------------------------------
def rope(v: np.ndarray, pos, theta: float, style: int = ROPE_HALF_SPLIT) -> np.ndarray:
    """Apply R_{Theta,pos} to the last axis (length d_h) of v.

    pos is a scalar or an array broadcastable to v.shape[:-1].  For j < d_h/2
    the pair (a, b) = (v[j], v[j + d_h/2]) [half split] or (v[2j], v[2j+1])
    [interleaved] is rotated by the angle pos * theta^(-2j/d_h):
        a' = a cos - b sin,   b' = a sin + b cos.
    Positions are 0-based.
    """
    v = np.asarray(v, dtype=np.float64)
    d = v.shape[-1]
    half = d // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = float(theta) ** (-2.0 * j / d)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(v)
    if style == ROPE_HALF_SPLIT:
        a, b = v[..., :half], v[..., half:]
        out[..., :half] = a * c - b * s
        out[..., half:] = a * s + b * c
    elif style == ROPE_INTERLEAVED:
        a, b = v[..., 0::2], v[..., 1::2]
        out[..., 0::2] = a * c - b * s
        out[..., 1::2] = a * s + b * c
    else:
        raise ValueError("unknown rope style")
    return out


# --------------------------------------------------------------------------
# attention (Preliminary section, Attention(Q,K,V) = softmax(Q K^T / sqrt(d_k)) V; Sec. 3.3 GQA repeat)
# --------------------------------------------------------------------------
def attention_one_query(q_hat: np.ndarray, K_hat: np.ndarray, V: np.ndarray) -> np.ndarray:
    """One decode query per head over N cached tokens.

    q_hat [H_q, d_h] (already rotated), K_hat [N, H_kv, d_h] (already rotated),
    V [N, H_kv, d_h].  Query head h uses KV head h // (H_q / H_kv): Sec. 3.3
    replicates each fetched KV head across the query heads of its group.
    Returns [H_q, d_h].
    """
    H_q, d = q_hat.shape
    N, H_kv, _ = K_hat.shape
    G = H_q // H_kv
    out = np.empty((H_q, d), dtype=np.float64)
    for h in range(H_q):
        g = h // G
        s = K_hat[:, g, :] @ q_hat[h] / math.sqrt(d)
        s = s - np.max(s)
        p = np.exp(s)
        p = p / np.sum(p)
        out[h] = p @ V[:, g, :]
    return out


def decode_attn_latent(c_k: np.ndarray, c_v: np.ndarray, B_k: np.ndarray, B_v: np.ndarray,
                       q: np.ndarray, n_kv_heads: int, theta: float,
                       style: int = ROPE_HALF_SPLIT, positions=None, q_position=None,
                       use_rope: bool = True) -> np.ndarray:
    """Decode attention of one sequence over its latent cache.

    c_k [N, r_k], c_v [N, r_v]: cached latents (whatever precision the cache held,
    passed as fp64).  B_k [r_k, n], B_v [r_v, n].  q [H_q, d_h] un-rotated.
    Steps, in the paper's order: fetch the compressed rows; reconstruct keys and
    values for all KV heads (K~ = C_K B_K, V~ = C_V B_V); rotate each key at its
    own position and the query at its position (Appendix "Adjusted Position
    Embedding"); attention with GQA repeat (Sec. 3.3).  By default the N cached
    tokens sit at positions 0..N-1 and the query at N-1 (the token appended last).
    """
    c_k = np.asarray(c_k, dtype=np.float64)
    c_v = np.asarray(c_v, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    N = c_k.shape[0]
    H_q, d = q.shape
    K = (c_k @ np.asarray(B_k, dtype=np.float64)).reshape(N, n_kv_heads, d)
    V = (c_v @ np.asarray(B_v, dtype=np.float64)).reshape(N, n_kv_heads, d)
    if positions is None:
        positions = np.arange(N)
    if q_position is None:
        q_position = N - 1
    if use_rope:
        K = rope(K, np.asarray(positions)[:, None], theta, style)
        q = rope(q, np.full((H_q,), q_position), theta, style)
    return attention_one_query(q, K, V)


def decode_attn_latent_out(c_k: np.ndarray, c_v: np.ndarray, B_k: np.ndarray, q: np.ndarray,
                           n_kv_heads: int, theta: float, style: int = ROPE_HALF_SPLIT,
                           use_rope: bool = True) -> np.ndarray:
    """Decode attention stopped before the value up-projection: o_lat[h] = sum_n p[h, n] c^V_n, [H_q, r_v].

    The probabilities are those of decode_attn_latent (keys reconstructed, rotated, softmax); the values are left
    as cached latents.  Sec. 3.1 (the W_o' equation) folds the remaining factor into the output projection:
    decode_attn_latent's output is o_lat[h] B_V[:, g(h)]."""
    c_k = np.asarray(c_k, dtype=np.float64)
    c_v = np.asarray(c_v, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    N = c_k.shape[0]
    H_q, d = q.shape
    G = H_q // n_kv_heads
    K = (c_k @ np.asarray(B_k, dtype=np.float64)).reshape(N, n_kv_heads, d)
    if use_rope:
        K = rope(K, np.arange(N)[:, None], theta, style)
        q = rope(q, np.full((H_q,), N - 1), theta, style)
    out = np.empty((H_q, c_v.shape[1]), dtype=np.float64)
    for h in range(H_q):
        s = K[:, h // G, :] @ q[h] / math.sqrt(d)
        p = np.exp(s - np.max(s))
        out[h] = (p / np.sum(p)) @ c_v
    return out


def prefill_attn_latent(c_k: np.ndarray, c_v: np.ndarray, B_k: np.ndarray, B_v: np.ndarray, q: np.ndarray,
                        n_kv_heads: int, theta: float, style: int = ROPE_HALF_SPLIT,
                        use_rope: bool = True) -> np.ndarray:
    """Attention of the T newest tokens of one sequence over its latent cache (prompt processing in chunks).

    c_k [N, r_k], c_v [N, r_v] hold ALL N cached tokens, the T new ones last; q [T, H_q, d_h] are their un-rotated
    queries.  Query t sits at position N - T + t and attends to the tokens at positions 0 .. N - T + t (the cached
    prefix in full, the new chunk causally): the Preliminary section's Attention(Q, K, V) with the usual causal mask,
    keys and values reconstructed from the latents as in decode_attn_latent.  Written as that function applied to
    each query with the cache cut after its own position.  Returns [T, H_q, d_h]."""
    q = np.asarray(q, dtype=np.float64)
    T = q.shape[0]
    N = np.asarray(c_k).shape[0]
    out = np.empty(q.shape, dtype=np.float64)
    for t in range(T):
        n_t = N - T + t + 1
        out[t] = decode_attn_latent(c_k[:n_t], c_v[:n_t], B_k, B_v, q[t], n_kv_heads, theta, style, use_rope=use_rope)
    return out


def shard_log2_sum_exp(c_k: np.ndarray, B_k: np.ndarray, q: np.ndarray, n_kv_heads: int, theta: float,
                        positions, q_position: int, style: int = ROPE_HALF_SPLIT, use_rope: bool = True) -> np.ndarray:
    """log2 of sum_n exp(s_n) per query head, over the cached rows given (a shard of one context).

    s_n = q^ . k^_n / sqrt(d_h) are the scores of the Preliminary section's attention with keys reconstructed and
    rotated at `positions` and the query rotated at q_position.  A softmax over a union of disjoint shards weights
    each shard's own softmax result by exp of this quantity; that is all a context-sharded decode has to exchange
    besides the shard outputs.  Returns [H_q] (-inf for an empty shard)."""
    c_k = np.asarray(c_k, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    N = c_k.shape[0]
    H_q, d = q.shape
    G = H_q // n_kv_heads
    if N == 0:
        return np.full((H_q,), -np.inf)
    K = (c_k @ np.asarray(B_k, dtype=np.float64)).reshape(N, n_kv_heads, d)
    if use_rope:
        K = rope(K, np.asarray(positions)[:, None], theta, style)
        q = rope(q, np.full((H_q,), q_position), theta, style)
    out = np.empty((H_q,), dtype=np.float64)
    for h in range(H_q):
        s = K[:, h // G, :] @ q[h] / math.sqrt(d)
        m = np.max(s)
        out[h] = (m + math.log(np.sum(np.exp(s - m)))) / math.log(2.0)
    return out


def merge_context_shards(outs: np.ndarray, log2_sums: np.ndarray) -> np.ndarray:
    """Attention over the union of disjoint shards from the shards' own results.

    outs [R, ..., d_h]: each shard's attention output (its own softmax); log2_sums [R, ...]: shard_log2_sum_exp.
    softmax over the union = sum_r w_r out_r / sum_r w_r with w_r = 2^(log2_sums_r): the denominators of the
    shards' softmaxes add up to the denominator of the whole.  Shards with -inf (no token) drop out."""
    outs = np.asarray(outs, dtype=np.float64)
    ls = np.asarray(log2_sums, dtype=np.float64)
    top = np.max(ls, axis=0)
    w = np.where(np.isfinite(ls), np.exp2(ls - np.where(np.isfinite(top), top, 0.0)), 0.0)
    return np.sum(w[..., None] * outs, axis=0) / np.sum(w, axis=0)[..., None]


def decode_attn_full(x: np.ndarray, W_k: np.ndarray, W_v: np.ndarray, q: np.ndarray,
                     n_kv_heads: int, theta: float, style: int = ROPE_HALF_SPLIT,
                     positions=None, q_position=None, use_rope: bool = True) -> np.ndarray:
    """Uncompressed decode attention: K = X W_k, V = X W_v, rotate, attend.

    x [N, D] are the hidden states of the N cached tokens.  This is the
    definition the compressed path must reproduce exactly at full rank.
    """
    x = np.asarray(x, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    N = x.shape[0]
    H_q, d = q.shape
    K = (x @ np.asarray(W_k, dtype=np.float64)).reshape(N, n_kv_heads, d)
    V = (x @ np.asarray(W_v, dtype=np.float64)).reshape(N, n_kv_heads, d)
    if positions is None:
        positions = np.arange(N)
    if q_position is None:
        q_position = N - 1
    if use_rope:
        K = rope(K, np.asarray(positions)[:, None], theta, style)
        q = rope(q, np.full((H_q,), q_position), theta, style)
    return attention_one_query(q, K, V)


def decode_attn_cached_kv(k_rot: np.ndarray, v: np.ndarray, q: np.ndarray, theta: float,
                          style: int = ROPE_HALF_SPLIT, q_position=None) -> np.ndarray:
    """Attention over an uncompressed cache that already holds rotated keys.

    k_rot, v [N, H_kv, d_h]; q [H_q, d_h] un-rotated, rotated here at q_position
    (default N-1).  This is the conventional pipeline the appendix contrasts
    with: an ordinary cache holds keys that were rotated before being stored.
    """
    k_rot = np.asarray(k_rot, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    N = k_rot.shape[0]
    if q_position is None:
        q_position = N - 1
    qh = rope(q, np.full((q.shape[0],), q_position), theta, style)
    return attention_one_query(qh, k_rot, np.asarray(v, dtype=np.float64))


# --------------------------------------------------------------------------
# batch / paged drivers (plain indexing around the functions above)
# --------------------------------------------------------------------------
def gather_rows(pool: np.ndarray, page_table_row: np.ndarray, length: int, page_size: int) -> np.ndarray:
    """Rows 0..length-1 of one sequence from a paged pool [n_pages, page_size, r]."""
    n_pg = (length + page_size - 1) // page_size
    rows = pool[np.asarray(page_table_row[:n_pg], dtype=np.int64)].reshape(n_pg * page_size, -1)
    return rows[:length]


def decode_attn_latent_batch(cache_k, cache_v, seq_lens, B_k, B_v, q, n_kv_heads, theta,
                             style=ROPE_HALF_SPLIT, page_table=None, page_size=64):
    """Loop of decode_attn_latent over a ragged batch.

    Contiguous: cache_* [b, N_max, r].  Paged: cache_* [n_pages, page_size, r] with
    page_table [b, max_pages].  q [b, H_q, d_h].  Returns [b, H_q, d_h].
    """
    b = len(seq_lens)
    out = np.empty(np.asarray(q).shape, dtype=np.float64)
    for s in range(b):
        L = int(seq_lens[s])
        if page_table is None:
            ck, cv = cache_k[s, :L], cache_v[s, :L]
        else:
            ck = gather_rows(cache_k, page_table[s], L, page_size)
            cv = gather_rows(cache_v, page_table[s], L, page_size)
        out[s] = decode_attn_latent(ck, cv, B_k, B_v, q[s], n_kv_heads, theta, style)
    return out


def rel_l2_rows(got: np.ndarray, want: np.ndarray) -> float:
    """max over rows (last axis = row) of ||got - want||_2 / ||want||_2."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    num = np.sqrt(np.sum((got - want) ** 2, axis=-1))
    den = np.sqrt(np.sum(want ** 2, axis=-1))
    den = np.where(den == 0.0, 1.0, den)
    return float(np.max(num / den))
