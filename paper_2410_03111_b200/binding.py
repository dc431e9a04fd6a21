"""ctypes binding of liblorc.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it calls
(see include/lorc.h).  Tensors are torch CUDA tensors (device memory) unless the
name says host; nothing is computed in Python.  Importing this module fails
loudly when the compiled library is missing: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "liblorc.so")

LORC_OK = 0
LORC_ERR_ARG = 1
LORC_ERR_LAYER = 2
LORC_ERR_CAPACITY = 3
LORC_ERR_EMPTY = 4
LORC_ERR_TIMEOUT = 5
LORC_ERR_CUDA = 6
LORC_ERR_UNSUPPORTED = 7
LORC_ERR_WORKSPACE = 8
LORC_MODE_LATENT = 0
LORC_MODE_FULL = 1
LORC_ROPE_HALF_SPLIT = 0
LORC_ROPE_INTERLEAVED = 1
LORC_ROPE_NONE = 2
LORC_FLAG_DEBUG_FP32 = 1
LORC_FLAG_PROFILE = 2
LORC_N_STAGES = 4
LORC_STAGE_NAMES = ("append", "score", "pv", "combine")
LORC_STATIC_SCRATCH_BYTES = 8 << 20


class lorc_model_desc(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("d_head", C.c_int32), ("rope_style", C.c_int32),
        ("max_pos", C.c_int32), ("flags", C.c_int32), ("rope_theta", C.c_double),
    ]


class lorc_cache(C.Structure):
    _fields_ = [
        ("k", C.c_void_p), ("v", C.c_void_p), ("page_table", C.c_void_p), ("seq_lens", C.c_void_p),
        ("batch", C.c_int32), ("max_seq_len", C.c_int32), ("page_size", C.c_int32),
        ("max_pages_per_seq", C.c_int32), ("n_pages", C.c_int32), ("reserved", C.c_int32),
        ("seq_stride", C.c_int64),
    ]


class LorcError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"lorc error {code}: {msg}")
        self.code = code


def _signatures():
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_int64
    cp = C.POINTER(lorc_cache)
    return {
        "lorc_create": ([C.POINTER(lorc_model_desc), C.POINTER(vp)], i32),
        "lorc_destroy": ([vp], i32),
        "lorc_load_factors": ([vp, i32, i32, i32, i32, vp, vp, vp, vp, vp], i32),
        "lorc_workspace_bytes": ([vp, i32, i32], C.c_size_t),
        "lorc_set_workspace": ([vp, vp, C.c_size_t], i32),
        "lorc_append": ([vp, i32, cp, vp, i32, vp], i32),
        "lorc_decode_attn": ([vp, i32, cp, vp, vp, i32, vp], i32),
        "lorc_decode_attn_latent_out": ([vp, i32, cp, vp, vp, i32, vp], i32),
        "lorc_prefill_workspace_bytes": ([vp, i32, i32, i32], C.c_size_t),
        "lorc_prefill_attn": ([vp, i32, cp, vp, vp, i32, vp], i32),
        "lorc_selftest_wait_expiry": ([vp, C.c_ulonglong, vp], i32),
        "lorc_decode_attn_shard": ([vp, i32, cp, vp, vp, vp, vp, vp, i32, vp], i32),
        "lorc_merge_shards": ([vp, i32, vp, vp, vp, i32, vp], i32),
        "lorc_decode_attn_static": ([vp, i32, cp, vp, vp, i32, vp], i32),
        "lorc_decode_step_host": ([vp, i32, cp, vp, vp, vp, i32, vp], i32),
        "lorc_sync_status": ([vp, vp], i32),
        "lorc_last_error": ([vp], C.c_char_p),
        "lorc_last_path": ([vp], i32),
        "lorc_profile_read": ([vp, C.POINTER(C.c_float), C.POINTER(i64)], i32),
        "lorc_profile_enable": ([vp, i32], i32),
        "lorc_launch_count": ([vp], i64),
    }


EXPORTS = sorted(_signatures())


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2410_03111_b200._build` "
            "(there is no non-CUDA fallback)")
    lib = C.CDLL(LIB_PATH)
    for name, (argtypes, restype) in _signatures().items():
        fn = getattr(lib, name)          # AttributeError if the symbol is missing
        fn.argtypes = argtypes
        fn.restype = restype
    return lib


_lib = _load()


def _ptr(t):
    """Device / host address of a torch tensor (or None, or a raw integer address)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(ctx, rc):
    if rc != LORC_OK:
        msg = _lib.lorc_last_error(ctx).decode() if ctx else "no context"
        raise LorcError(rc, msg)


def lorc_create(n_layers, d_model, n_q_heads, n_kv_heads, d_head, rope_theta,
                rope_style=LORC_ROPE_HALF_SPLIT, max_pos=4096, flags=0):
    desc = lorc_model_desc(n_layers, d_model, n_q_heads, n_kv_heads, d_head, rope_style, max_pos, flags,
                           float(rope_theta))
    out = C.c_void_p()
    rc = _lib.lorc_create(C.byref(desc), C.byref(out))
    if rc != LORC_OK:
        raise LorcError(rc, "lorc_create failed")
    return out


def lorc_destroy(ctx):
    _check(None, _lib.lorc_destroy(ctx))


def lorc_load_factors(ctx, layer, mode, r_k, r_v, A_k, B_k, A_v, B_v, stream=None):
    _check(ctx, _lib.lorc_load_factors(ctx, layer, mode, r_k, r_v, _ptr(A_k), _ptr(B_k), _ptr(A_v),
                                        _ptr(B_v), _stream(stream)))


def lorc_workspace_bytes(ctx, batch, max_seq_len):
    return int(_lib.lorc_workspace_bytes(ctx, batch, max_seq_len))


def lorc_set_workspace(ctx, workspace, nbytes=None):
    if workspace is None:
        _check(ctx, _lib.lorc_set_workspace(ctx, None, 0))
        return
    if nbytes is None:
        nbytes = workspace.numel() * workspace.element_size()
    _check(ctx, _lib.lorc_set_workspace(ctx, _ptr(workspace), nbytes))


def make_cache(k, v, seq_lens, batch, max_seq_len, page_table=None, page_size=0, max_pages_per_seq=0,
               n_pages=0, seq_stride=0):
    """Fill a lorc_cache descriptor from tensors (pointers only; nothing is copied)."""
    return lorc_cache(_ptr(k), _ptr(v), _ptr(page_table), _ptr(seq_lens), batch, max_seq_len, page_size,
                      max_pages_per_seq, n_pages, 0, seq_stride)


def lorc_append(ctx, layer, cache, x, T=1, stream=None):
    _check(ctx, _lib.lorc_append(ctx, layer, C.byref(cache), _ptr(x), T, _stream(stream)))


def lorc_decode_attn(ctx, layer, cache, q, out, n_splits=0, stream=None):
    _check(ctx, _lib.lorc_decode_attn(ctx, layer, C.byref(cache), _ptr(q), _ptr(out), n_splits,
                                       _stream(stream)))


def lorc_prefill_workspace_bytes(ctx, batch, max_seq_len, T):
    return int(_lib.lorc_prefill_workspace_bytes(ctx, batch, max_seq_len, T))


def lorc_prefill_attn(ctx, layer, cache, q, out, T, stream=None):
    _check(ctx, _lib.lorc_prefill_attn(ctx, layer, C.byref(cache), _ptr(q), _ptr(out), T, _stream(stream)))


def lorc_decode_attn_latent_out(ctx, layer, cache, q, o_lat, n_splits=0, stream=None):
    _check(ctx, _lib.lorc_decode_attn_latent_out(ctx, layer, C.byref(cache), _ptr(q), _ptr(o_lat), n_splits,
                                                  _stream(stream)))


def lorc_decode_attn_shard(ctx, layer, cache, q, pos0, q_pos, out, ml, n_splits=0, stream=None):
    _check(ctx, _lib.lorc_decode_attn_shard(ctx, layer, C.byref(cache), _ptr(q), _ptr(pos0), _ptr(q_pos), _ptr(out),
                                             _ptr(ml), n_splits, _stream(stream)))


def lorc_merge_shards(ctx, n_shards, outs, mls, out, batch, stream=None):
    _check(ctx, _lib.lorc_merge_shards(ctx, n_shards, _ptr(outs), _ptr(mls), _ptr(out), batch, _stream(stream)))


def lorc_decode_attn_static(ctx, layer, cache, q, out, n_splits=0, stream=None):
    """lorc_decode_attn for callers that cannot allocate: scratch is a fixed array in the library."""
    _check(ctx, _lib.lorc_decode_attn_static(ctx, layer, C.byref(cache), _ptr(q), _ptr(out), n_splits,
                                              _stream(stream)))


def lorc_decode_step_host(ctx, layer, cache, x_host, q_host, out_host, n_splits=0, stream=None):
    _check(ctx, _lib.lorc_decode_step_host(ctx, layer, C.byref(cache), _ptr(x_host), _ptr(q_host),
                                            _ptr(out_host), n_splits, _stream(stream)))


def lorc_selftest_wait_expiry(ctx, limit_ns, stream=None):
    _check(ctx, _lib.lorc_selftest_wait_expiry(ctx, int(limit_ns), _stream(stream)))


def lorc_sync_status(ctx, stream=None):
    return int(_lib.lorc_sync_status(ctx, _stream(stream)))


def lorc_last_error(ctx):
    return _lib.lorc_last_error(ctx).decode()


def lorc_last_path(ctx):
    return int(_lib.lorc_last_path(ctx))


def lorc_profile_read(ctx):
    """Device milliseconds and launch counts per stage since the last call (LORC_FLAG_PROFILE contexts)."""
    ms = (C.c_float * LORC_N_STAGES)()
    cnt = (C.c_int64 * LORC_N_STAGES)()
    _check(ctx, _lib.lorc_profile_read(ctx, ms, cnt))
    return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(LORC_STAGE_NAMES)}


def lorc_profile_enable(ctx, on):
    """Turn the per-stage event bracketing on or off for the calls that follow."""
    _check(ctx, _lib.lorc_profile_enable(ctx, 1 if on else 0))


def lorc_launch_count(ctx):
    return int(_lib.lorc_launch_count(ctx))
