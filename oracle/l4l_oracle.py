"""ctypes front end of the CPU oracle (``l4l_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module. It shares no code with the CUDA
path. All arithmetic lives in the C file; this file only builds it with gcc, turns
arrays into pointers and allocates the fp64 outputs.

Inputs are bf16 given either as ``torch.bfloat16`` CPU tensors or as numpy ``uint16``
arrays of the raw bits; outputs are numpy ``float64`` (caches: ``uint16`` bits).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "l4l_oracle.c")
_LIB = os.path.join(_HERE, "libl4l_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP); returns the path of the library."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        i, d = ctypes.c_int, ctypes.c_double
        lib.l4l_oracle_num_threads.restype = i
        lib.l4l_oracle_prefill.argtypes = [u16p, u16p, u16p, i32p, i, i, i, i, i, d, f64p, f64p]
        lib.l4l_oracle_prefill_rows.argtypes = [u16p, u16p, u16p, i32p, i, i, i, i, i, d,
                                                i32p, i, f64p, f64p]
        lib.l4l_oracle_decode.argtypes = [u16p, u16p, u16p, i32p, i, i, i, i, i, d, f64p, f64p]
        lib.l4l_oracle_prefill_chunk.argtypes = [u16p, u16p, u16p, i32p, i32p, i, i, i, i, i, i, d, f64p, f64p]
        f32p = ctypes.POINTER(ctypes.c_float)
        lib.l4l_oracle_round_bf16.argtypes = [f64p, u16p, ctypes.c_int64]
        lib.l4l_oracle_round_bf16.restype = None
        lib.l4l_oracle_rope_kv_append.argtypes = [u16p, u16p, u16p, u16p, u16p, i32p, i32p, i, i, i, i, i, i,
                                                  f32p, f32p, i, f32p, f32p, d, f64p, f64p]
        u8p = ctypes.POINTER(ctypes.c_uint8)
        lib.l4l_oracle_e4m3_decode.argtypes = [u8p, f64p, ctypes.c_int64]
        lib.l4l_oracle_e4m3_decode.restype = None
        lib.l4l_oracle_e4m3_encode.argtypes = [f32p, u8p, ctypes.c_int64]
        lib.l4l_oracle_e4m3_encode.restype = None
        lib.l4l_oracle_kv_append_fp8.argtypes = [u8p, u8p, u16p, u16p, i32p, i32p, f32p, f32p, i, i, i, i, i]
        lib.l4l_oracle_decode_fp8.argtypes = [u16p, u8p, u8p, i32p, f32p, f32p, i, i, i, i, i, d, f64p, f64p]
        lib.l4l_oracle_rglru.argtypes = [u16p, u16p, u16p, f32p, i32p, i32p, f64p, f64p, i, i, i]
        lib.l4l_oracle_kv_append.argtypes = [u16p, u16p, u16p, u16p, i32p, i32p, i, i, i, i, i]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().l4l_oracle_num_threads())


def bits(x) -> np.ndarray:
    """Raw bf16 bits as a C-contiguous uint16 array (accepts torch.bfloat16 or uint16)."""
    if isinstance(x, np.ndarray):
        if x.dtype != np.uint16:
            raise TypeError("numpy input must be uint16 bf16 bits")
        return np.ascontiguousarray(x)
    import torch  # device memory / tensor container only

    if x.dtype != torch.bfloat16:
        raise TypeError("tensor input must be bfloat16")
    return np.ascontiguousarray(x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def _p(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def _i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def prefill(q, k, v, seq_len, scale: float):
    """Causal prefill. q [B,S,Hq,D], k/v [B,S,Hkv,D]; returns (out [B,S,Hq,D], lse [B,Hq,S]).

    Rows i >= seq_len[b] are NaN in both outputs (they are not defined)."""
    q, k, v = bits(q), bits(k), bits(v)
    B, S, Hq, D = q.shape
    Hkv = k.shape[2]
    assert k.shape == (B, S, Hkv, D) and v.shape == k.shape
    sl = _i32(seq_len)
    assert sl.shape == (B,) and (sl >= 0).all() and (sl <= S).all()
    out = np.full((B, S, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, Hq, S), np.nan, dtype=np.float64)
    rc = _load().l4l_oracle_prefill(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                                    _p(v, ctypes.c_uint16), _p(sl, ctypes.c_int32),
                                    B, S, Hq, Hkv, D, float(scale),
                                    _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_prefill rejected its arguments")
    return out, lse


def prefill_rows(q, k, v, seq_len, scale: float, rows):
    """Causal prefill of the listed (b, i, h) rows only; returns (out [n,D], lse [n])."""
    q, k, v = bits(q), bits(k), bits(v)
    B, S, Hq, D = q.shape
    Hkv = k.shape[2]
    sl = _i32(seq_len)
    rows = _i32(rows).reshape(-1, 3)
    n = rows.shape[0]
    out = np.empty((n, D), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    rc = _load().l4l_oracle_prefill_rows(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                                         _p(v, ctypes.c_uint16), _p(sl, ctypes.c_int32),
                                         B, S, Hq, Hkv, D, float(scale),
                                         _p(rows, ctypes.c_int32), n,
                                         _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_prefill_rows rejected its arguments")
    return out, lse


def prefill_chunk(q, cache_k, cache_v, past, q_len, scale: float):
    """Chunk of new tokens over a populated cache. q [B,S,Hq,D], caches [B,Hkv,Lmax,D] already holding the
    chunk's K/V at slots past..past+q_len-1; returns (out [B,S,Hq,D], lse [B,Hq,S]), NaN in undefined rows."""
    q, ck, cv = bits(q), bits(cache_k), bits(cache_v)
    B, S, Hq, D = q.shape
    _, Hkv, Lmax, _ = ck.shape
    assert ck.shape == (B, Hkv, Lmax, D) and cv.shape == ck.shape
    past, q_len = _i32(past), _i32(q_len)
    out = np.full((B, S, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((B, Hq, S), np.nan, dtype=np.float64)
    rc = _load().l4l_oracle_prefill_chunk(_p(q, ctypes.c_uint16), _p(ck, ctypes.c_uint16), _p(cv, ctypes.c_uint16),
                                          _p(past, ctypes.c_int32), _p(q_len, ctypes.c_int32), B, S, Hq, Hkv, D,
                                          Lmax, float(scale), _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_prefill_chunk rejected its arguments")
    return out, lse


def decode(q, cache_k, cache_v, kv_len, scale: float):
    """Decode. q [B,Hq,D], caches [B,Hkv,Lmax,D]; returns (out [B,Hq,D], lse [B,Hq])."""
    q, ck, cv = bits(q), bits(cache_k), bits(cache_v)
    B, Hq, D = q.shape
    _, Hkv, Lmax, _ = ck.shape
    assert ck.shape == (B, Hkv, Lmax, D) and cv.shape == ck.shape
    kl = _i32(kv_len)
    assert kl.shape == (B,) and (kl >= 0).all() and (kl <= Lmax).all()
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = _load().l4l_oracle_decode(_p(q, ctypes.c_uint16), _p(ck, ctypes.c_uint16),
                                   _p(cv, ctypes.c_uint16), _p(kl, ctypes.c_int32),
                                   B, Hq, Hkv, D, Lmax, float(scale),
                                   _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_decode rejected its arguments")
    return out, lse


def kv_append(cache_k, cache_v, k_new, v_new, pos, n_new):
    """Returns copies of the caches (uint16 bits) with the new tokens written in."""
    ck, cv = bits(cache_k).copy(), bits(cache_v).copy()
    kn, vn = bits(k_new), bits(v_new)
    B, Hkv, Lmax, D = ck.shape
    T = kn.shape[1]
    assert kn.shape == (B, T, Hkv, D) and vn.shape == kn.shape
    pos, n_new = _i32(pos), _i32(n_new)
    rc = _load().l4l_oracle_kv_append(_p(ck, ctypes.c_uint16), _p(cv, ctypes.c_uint16),
                                      _p(kn, ctypes.c_uint16), _p(vn, ctypes.c_uint16),
                                      _p(pos, ctypes.c_int32), _p(n_new, ctypes.c_int32),
                                      B, T, Hkv, D, Lmax)
    if rc != 0:
        raise ValueError("l4l_oracle_kv_append: write outside the cache")
    return ck, cv


def round_bf16(x) -> np.ndarray:
    """fp64 array -> bf16 bits (uint16), round to nearest even."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    out = np.empty(x.shape, dtype=np.uint16)
    _load().l4l_oracle_round_bf16(_p(x, ctypes.c_double), _p(out, ctypes.c_uint16), x.size)
    return out


def rope_kv_append(q, k_new, v_new, cache_k, cache_v, pos, n_new, cos, sin, q_weight=None, k_weight=None,
                   eps: float = 0.0):
    """Rotary embedding (+ optional RMS norm) of q and k fused with the cache update.

    q [B,T,Hq,D], k_new/v_new [B,T,Hkv,D], caches [B,Hkv,Lmax,D], cos/sin float32 [n_pos, D/2].
    Returns (q_bits, cache_k_bits, cache_v_bits, q_exact, k_exact): the first three as uint16 bf16 bits after
    the update, the last two the unrounded fp64 rotations (NaN in skipped rows)."""
    qb, kn, vn = bits(q).copy(), bits(k_new), bits(v_new)
    ck, cv = bits(cache_k).copy(), bits(cache_v).copy()
    B, T, Hq, D = qb.shape
    Hkv, Lmax = ck.shape[1], ck.shape[2]
    assert kn.shape == (B, T, Hkv, D) and vn.shape == kn.shape and ck.shape == (B, Hkv, Lmax, D)
    cos = np.ascontiguousarray(np.asarray(cos, dtype=np.float32))
    sin = np.ascontiguousarray(np.asarray(sin, dtype=np.float32))
    assert cos.shape == sin.shape and cos.shape[1] == D // 2
    pos = _i32(pos)
    n_new = _i32(n_new) if n_new is not None else np.full((B,), T, np.int32)
    f32 = ctypes.c_float
    qw = None if q_weight is None else np.ascontiguousarray(np.asarray(q_weight, dtype=np.float32))
    kw = None if k_weight is None else np.ascontiguousarray(np.asarray(k_weight, dtype=np.float32))
    q_exact = np.full(qb.shape, np.nan)
    k_exact = np.full(kn.shape, np.nan)
    rc = _load().l4l_oracle_rope_kv_append(
        _p(qb, ctypes.c_uint16), _p(kn, ctypes.c_uint16), _p(vn, ctypes.c_uint16), _p(ck, ctypes.c_uint16),
        _p(cv, ctypes.c_uint16), _p(pos, ctypes.c_int32), _p(n_new, ctypes.c_int32), B, T, Hq, Hkv, D, Lmax,
        _p(cos, f32), _p(sin, f32), cos.shape[0], None if qw is None else _p(qw, f32),
        None if kw is None else _p(kw, f32), float(eps), _p(q_exact, ctypes.c_double), _p(k_exact, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_rope_kv_append rejected its arguments")
    return qb, ck, cv, q_exact, k_exact


def gather_pages(pool, block_table, n_slots: int) -> np.ndarray:
    """Paged cache -> the contiguous cache it stands for. pool [pages, Hkv, page_size, D] (bf16 bits or tensor),
    block_table [B, n] ints; returns uint16 [B, Hkv, n_slots, D]: slot s of sequence b is row s % page_size of page
    block_table[b, s // page_size]. Entries outside the pool read as zeros (as the GPU path defines)."""
    pb = bits(pool)
    n_pages, Hkv, page, D = pb.shape
    bt = np.asarray(block_table, dtype=np.int64)
    B = bt.shape[0]
    out = np.zeros((B, Hkv, n_slots, D), dtype=np.uint16)
    for b in range(B):
        for s0 in range(0, n_slots, page):
            pg = bt[b, s0 // page] if s0 // page < bt.shape[1] else -1
            if 0 <= pg < n_pages:
                n = min(page, n_slots - s0)
                out[b, :, s0:s0 + n] = pb[pg, :, :n]
    return out


def decode_paged(q, pool_k, pool_v, block_table, kv_len, scale: float):
    """Decode over a paged cache = decode over the gathered contiguous cache."""
    kl = _i32(kv_len)
    n_slots = max(int(kl.max()) if kl.size else 0, 1)
    return decode(q, gather_pages(pool_k, block_table, n_slots), gather_pages(pool_v, block_table, n_slots), kl, scale)


def kv_append_paged(pool_k, pool_v, block_table, k_new, v_new, pos, n_new):
    """Returns copies of the pools (uint16 bits) with the new tokens written to their pages."""
    pk, pv = bits(pool_k).copy(), bits(pool_v).copy()
    kn, vn = bits(k_new), bits(v_new)
    n_pages, Hkv, page, D = pk.shape
    bt = np.asarray(block_table, dtype=np.int64)
    B, T = kn.shape[0], kn.shape[1]
    pos = _i32(pos)
    n_new = _i32(n_new) if n_new is not None else np.full((B,), T, np.int32)
    for b in range(B):
        for t in range(min(T, int(n_new[b]))):
            s = int(pos[b]) + t
            if s < 0 or s // page >= bt.shape[1]:
                continue
            pg = bt[b, s // page]
            if 0 <= pg < n_pages:
                pk[pg, :, s % page] = kn[b, t]
                pv[pg, :, s % page] = vn[b, t]
    return pk, pv


def _u8(x) -> np.ndarray:
    """uint8 codes from a numpy uint8 array or a torch uint8 / float8_e4m3fn tensor."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint8
        return np.ascontiguousarray(x)
    import torch

    if x.dtype != torch.uint8:
        x = x.view(torch.uint8)
    return np.ascontiguousarray(x.detach().cpu().contiguous().numpy())


def e4m3_decode(codes) -> np.ndarray:
    c = _u8(codes)
    out = np.empty(c.shape, dtype=np.float64)
    _load().l4l_oracle_e4m3_decode(_p(c, ctypes.c_uint8), _p(out, ctypes.c_double), c.size)
    return out


def e4m3_encode(x) -> np.ndarray:
    """float32 values -> e4m3 codes (nearest even, saturating)."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    out = np.empty(x.shape, dtype=np.uint8)
    _load().l4l_oracle_e4m3_encode(_p(x, ctypes.c_float), _p(out, ctypes.c_uint8), x.size)
    return out


def kv_append_fp8(cache_k8, cache_v8, k_new, v_new, pos, n_new, k_scale, v_scale):
    """Returns copies of the fp8 caches (uint8 codes) with the new tokens quantised in."""
    ck, cv = _u8(cache_k8).copy(), _u8(cache_v8).copy()
    kn, vn = bits(k_new), bits(v_new)
    B, Hkv, Lmax, D = ck.shape
    T = kn.shape[1]
    assert kn.shape == (B, T, Hkv, D) and vn.shape == kn.shape
    pos = _i32(pos)
    n_new = _i32(n_new) if n_new is not None else np.full((B,), T, np.int32)
    ks = np.ascontiguousarray(np.asarray(k_scale, dtype=np.float32))
    vs = np.ascontiguousarray(np.asarray(v_scale, dtype=np.float32))
    assert ks.shape == (Hkv,) and vs.shape == (Hkv,)
    _load().l4l_oracle_kv_append_fp8(_p(ck, ctypes.c_uint8), _p(cv, ctypes.c_uint8), _p(kn, ctypes.c_uint16),
                                     _p(vn, ctypes.c_uint16), _p(pos, ctypes.c_int32), _p(n_new, ctypes.c_int32),
                                     _p(ks, ctypes.c_float), _p(vs, ctypes.c_float), B, T, Hkv, D, Lmax)
    return ck, cv


def decode_fp8(q, cache_k8, cache_v8, kv_len, k_scale, v_scale, scale: float):
    """Decode over an fp8 cache. q [B,Hq,D] bf16; caches [B,Hkv,Lmax,D] e4m3 codes; scales float32 [Hkv]."""
    q, ck, cv = bits(q), _u8(cache_k8), _u8(cache_v8)
    B, Hq, D = q.shape
    _, Hkv, Lmax, _ = ck.shape
    kl = _i32(kv_len)
    ks = np.ascontiguousarray(np.asarray(k_scale, dtype=np.float32))
    vs = np.ascontiguousarray(np.asarray(v_scale, dtype=np.float32))
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = _load().l4l_oracle_decode_fp8(_p(q, ctypes.c_uint16), _p(ck, ctypes.c_uint8), _p(cv, ctypes.c_uint8),
                                       _p(kl, ctypes.c_int32), _p(ks, ctypes.c_float), _p(vs, ctypes.c_float),
                                       B, Hq, Hkv, D, Lmax, float(scale), _p(out, ctypes.c_double),
                                       _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("l4l_oracle_decode_fp8 rejected its arguments")
    return out, lse


def rglru(x, gate_x, gate_a, a_param, state=None, position=None, seq_len=None):
    """Gated linear recurrence (RG-LRU). x, gate_x, gate_a bf16 [B,T,W]; a_param float32 [W]; state fp64 [B,W] or
    None (zeros); position int32 [B,T] or None; seq_len [B] or None. Returns (y fp64 [B,T,W] with NaN in rows past
    seq_len, final state fp64 [B,W])."""
    xb, gx, ga = bits(x), bits(gate_x), bits(gate_a)
    B, T, W = xb.shape
    assert gx.shape == xb.shape and ga.shape == xb.shape
    ap = np.ascontiguousarray(np.asarray(a_param, dtype=np.float32))
    assert ap.shape == (W,)
    st = np.zeros((B, W)) if state is None else np.ascontiguousarray(np.asarray(state, dtype=np.float64)).copy()
    pos = None if position is None else _i32(position)
    sl = None if seq_len is None else _i32(seq_len)
    y = np.full((B, T, W), np.nan)
    rc = _load().l4l_oracle_rglru(_p(xb, ctypes.c_uint16), _p(gx, ctypes.c_uint16), _p(ga, ctypes.c_uint16),
                                  _p(ap, ctypes.c_float), None if pos is None else _p(pos, ctypes.c_int32),
                                  None if sl is None else _p(sl, ctypes.c_int32), _p(st, ctypes.c_double),
                                  _p(y, ctypes.c_double), B, T, W)
    if rc != 0:
        raise ValueError("l4l_oracle_rglru rejected its arguments")
    return y, st
