"""ctypes front end of the fp64 C oracle (`cq_oracle.c`) -- test infrastructure.

Arrays are numpy; fp16 inputs are passed as their bit patterns, codes as int32
in plain row-major order (the oracle knows nothing of the CUDA library's code
layout).  `build()` compiles the C file with gcc next to this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cq_oracle.c")
_LIB = os.path.join(_HERE, "libcq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent items)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        vp, i64, i32, f64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_set_num_threads.argtypes = [i32]
        L.oracle_encode.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, vp, vp]
        L.oracle_code_distance.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp]
        L.oracle_dequant.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp]
        L.oracle_decode_dense.argtypes = [vp, vp, vp, vp, vp, vp, f64, i32, i32, i32, i32, i32, i32, i64, vp]
        L.oracle_decode_lut.argtypes = [vp, vp, vp, vp, vp, vp, f64, i32, i32, i32, i32, i32, i32, i64, i32, vp]
        L.oracle_decode_dense_rope.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, f64, i32, i32, i32, i32, i32, i32, i64, vp]
        L.oracle_decode_dense_rope.restype = None
        L.oracle_prefill_dense.argtypes = [vp, vp, vp, vp, vp, vp, f64, i32, i32, i32, i32, i32, i32, i32, i64, vp]
        L.oracle_prefill_dense.restype = None
        L.oracle_kmeanspp_init.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp]
        L.oracle_lloyd_step.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, vp]
        L.oracle_kmeanspp_init.restype = None
        L.oracle_lloyd_step.restype = None
        for f in (L.oracle_set_num_threads, L.oracle_encode, L.oracle_code_distance, L.oracle_dequant,
                  L.oracle_decode_dense, L.oracle_decode_lut):
            f.restype = None
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _half_bits(x) -> np.ndarray:
    x = np.ascontiguousarray(x)
    if x.dtype == np.float16:
        return x.view(np.uint16)
    if x.dtype == np.uint16:
        return x
    raise TypeError("fp16 input expected (float16 array or its uint16 bit patterns)")


def _cb(cb, n_heads: int, D: int, c: int, b: int) -> np.ndarray:
    cb = np.ascontiguousarray(cb, dtype=np.float32)
    want = (n_heads, D // c, 1 << b, c)
    if cb.shape != want:
        raise ValueError(f"codebooks shape {cb.shape}, expected {want}")
    return cb


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def encode(x, codebooks, c: int, b: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """x fp16 (n_vec, n_heads, D), codebooks fp32 (n_heads, G, 2^b, c) ->
    (codes int32 (n_vec, n_heads, G), d_best fp64, d_second fp64)."""
    xb = _half_bits(x)
    n_vec, n_heads, D = xb.shape
    if D % c:
        raise ValueError("c must divide head_dim")
    cb = _cb(codebooks, n_heads, D, c, b)
    G = D // c
    codes = np.empty((n_vec, n_heads, G), dtype=np.int32)
    d1 = np.empty((n_vec, n_heads, G), dtype=np.float64)
    d2 = np.empty((n_vec, n_heads, G), dtype=np.float64)
    _load().oracle_encode(_p(xb), _p(cb), n_vec, n_heads, D, c, b, _p(codes), _p(d1), _p(d2))
    return codes, d1, d2


def code_distance(x, codebooks, codes, c: int, b: int) -> np.ndarray:
    """Squared distance of every group of x to the centroid named by `codes`."""
    xb = _half_bits(x)
    n_vec, n_heads, D = xb.shape
    cb = _cb(codebooks, n_heads, D, c, b)
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    assert codes.shape == (n_vec, n_heads, D // c)
    assert codes.min(initial=0) >= 0 and codes.max(initial=0) < (1 << b)
    out = np.empty(codes.shape, dtype=np.float64)
    _load().oracle_code_distance(_p(xb), _p(cb), _p(codes), n_vec, n_heads, D, c, b, _p(out))
    return out


def dequant(codes, codebooks, c: int, b: int) -> np.ndarray:
    """codes int32 (n_vec, n_heads, G) -> reconstruction fp64 (n_vec, n_heads, D)."""
    codes = np.ascontiguousarray(codes, dtype=np.int32)
    n_vec, n_heads, G = codes.shape
    D = G * c
    cb = _cb(codebooks, n_heads, D, c, b)
    assert codes.min(initial=0) >= 0 and codes.max(initial=0) < (1 << b)
    out = np.empty((n_vec, n_heads, D), dtype=np.float64)
    _load().oracle_dequant(_p(codes), _p(cb), n_vec, n_heads, D, c, b, _p(out))
    return out


def _attn_args(q, k_codes, v_codes, k_cb, v_cb, seq_lens, c, b):
    qb = _half_bits(q)
    n_seq, n_q_heads, D = qb.shape
    k_codes = np.ascontiguousarray(k_codes, dtype=np.int32)
    v_codes = np.ascontiguousarray(v_codes, dtype=np.int32)
    _, max_tokens, n_kv_heads, G = k_codes.shape
    assert k_codes.shape == v_codes.shape == (n_seq, max_tokens, n_kv_heads, D // c)
    assert n_q_heads % n_kv_heads == 0
    for cd in (k_codes, v_codes):
        assert cd.min(initial=0) >= 0 and cd.max(initial=0) < (1 << b)
    kcb = _cb(k_cb, n_kv_heads, D, c, b)
    vcb = _cb(v_cb, n_kv_heads, D, c, b)
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    assert sl.shape == (n_seq,) and sl.min(initial=0) >= 0 and sl.max(initial=0) <= max_tokens
    out = np.empty((n_seq, n_q_heads, D), dtype=np.float64)
    return qb, k_codes, v_codes, kcb, vcb, sl, n_seq, n_q_heads, n_kv_heads, D, max_tokens, out


def decode_dense(q, k_codes, v_codes, k_cb, v_cb, seq_lens, scale: float, c: int, b: int) -> np.ndarray:
    """Dequantise-then-softmax attention.  q fp16 (n_seq, Hq, D); codes int32
    (n_seq, max_tokens, Hkv, G); returns fp64 (n_seq, Hq, D)."""
    qb, kc, vc, kcb, vcb, sl, n_seq, hq, hkv, D, mt, out = _attn_args(q, k_codes, v_codes, k_cb, v_cb, seq_lens, c, b)
    _load().oracle_decode_dense(_p(qb), _p(kc), _p(vc), _p(kcb), _p(vcb), _p(sl), float(scale),
                                n_seq, hq, hkv, D, c, b, mt, _p(out))
    return out


def prefill_dense(q, k_codes, v_codes, k_cb, v_cb, seq_lens, scale: float, c: int, b: int) -> np.ndarray:
    """Causal attention of the last n_q cached tokens of every sequence.  q fp16 (n_seq, n_q, Hq, D);
    codes int32 (n_seq, max_tokens, Hkv, G); seq_lens counts the cached tokens including the n_q new
    ones; query i attends tokens 0 .. seq_lens[s] - n_q + i.  Returns fp64 (n_seq, n_q, Hq, D)."""
    qb = _half_bits(q)
    n_seq, n_q, n_q_heads, D = qb.shape
    k_codes = np.ascontiguousarray(k_codes, dtype=np.int32)
    v_codes = np.ascontiguousarray(v_codes, dtype=np.int32)
    _, max_tokens, n_kv_heads, G = k_codes.shape
    assert k_codes.shape == v_codes.shape == (n_seq, max_tokens, n_kv_heads, D // c)
    assert n_q_heads % n_kv_heads == 0
    for cd in (k_codes, v_codes):
        assert cd.min(initial=0) >= 0 and cd.max(initial=0) < (1 << b)
    kcb = _cb(k_cb, n_kv_heads, D, c, b)
    vcb = _cb(v_cb, n_kv_heads, D, c, b)
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    assert sl.shape == (n_seq,) and sl.min(initial=0) >= 0 and sl.max(initial=0) <= max_tokens
    out = np.empty((n_seq, n_q, n_q_heads, D), dtype=np.float64)
    _load().oracle_prefill_dense(_p(qb), _p(k_codes), _p(v_codes), _p(kcb), _p(vcb), _p(sl), float(scale),
                                 n_seq, n_q, n_q_heads, n_kv_heads, D, c, b, max_tokens, _p(out))
    return out


def decode_dense_rope(q, k_codes, v_codes, k_cb, v_cb, seq_lens, rope_cos, rope_sin, scale: float, c: int, b: int,
                      pairing: int = 0) -> np.ndarray:
    """Attention over codes of pre-RoPE keys: every reconstructed key is rotated by its position
    before the dot product.  rope_cos / rope_sin fp32 (max_tokens, D/2); pairing 0 = (i, i + D/2),
    1 = (2i, 2i + 1).  Returns fp64 (n_seq, Hq, D)."""
    qb, kc, vc, kcb, vcb, sl, n_seq, hq, hkv, D, mt, out = _attn_args(q, k_codes, v_codes, k_cb, v_cb, seq_lens, c, b)
    cs = np.ascontiguousarray(rope_cos, dtype=np.float32)
    sn = np.ascontiguousarray(rope_sin, dtype=np.float32)
    assert cs.shape == sn.shape == (mt, D // 2) and pairing in (0, 1) and D % 2 == 0
    _load().oracle_decode_dense_rope(_p(qb), _p(kc), _p(vc), _p(kcb), _p(vcb), _p(sl), _p(cs), _p(sn), int(pairing),
                                     float(scale), n_seq, hq, hkv, D, c, b, mt, _p(out))
    return out


def decode_lut(q, k_codes, v_codes, k_cb, v_cb, seq_lens, scale: float, c: int, b: int,
               n_chunks: int = 1) -> np.ndarray:
    """Same result through lookup tables, V bins and a chunked online softmax."""
    qb, kc, vc, kcb, vcb, sl, n_seq, hq, hkv, D, mt, out = _attn_args(q, k_codes, v_codes, k_cb, v_cb, seq_lens, c, b)
    _load().oracle_decode_lut(_p(qb), _p(kc), _p(vc), _p(kcb), _p(vcb), _p(sl), float(scale),
                              n_seq, hq, hkv, D, c, b, mt, int(n_chunks), _p(out))
    return out


def _weights(weights, n_vec, n_heads, G):
    if weights is None:
        return None
    w = np.ascontiguousarray(weights, dtype=np.float32)
    if w.shape != (n_vec, n_heads, G):
        raise ValueError(f"weights shape {w.shape}, expected {(n_vec, n_heads, G)}")
    assert (w >= 0).all()
    return w


def kmeanspp_init(x, weights, uniforms, c: int, b: int):
    """k-means++ with the draws passed in.  x fp16 (n_vec, n_heads, D); weights fp32
    (n_vec, n_heads, G) or None; uniforms fp64 (n_heads, G, 2^b) in [0, 1).
    Returns (codebooks fp32 (n_heads, G, 2^b, c), chosen int64 (n_heads, G, 2^b))."""
    xb = _half_bits(x)
    n_vec, n_heads, D = xb.shape
    G, K = D // c, 1 << b
    w = _weights(weights, n_vec, n_heads, G)
    u = np.ascontiguousarray(uniforms, dtype=np.float64)
    assert u.shape == (n_heads, G, K) and (u >= 0).all() and (u < 1).all()
    cb = np.empty((n_heads, G, K, c), dtype=np.float32)
    chosen = np.empty((n_heads, G, K), dtype=np.int64)
    _load().oracle_kmeanspp_init(_p(xb), _p(w), _p(u), n_vec, n_heads, D, c, b, _p(cb), _p(chosen))
    return cb, chosen


def lloyd_step(x, weights, codebooks, c: int, b: int):
    """One k-means iteration.  Returns (new codebooks fp32, codes int32 (n_vec, n_heads, G),
    objective fp64 (n_heads, G) of the assignment under the input codebooks)."""
    xb = _half_bits(x)
    n_vec, n_heads, D = xb.shape
    G = D // c
    w = _weights(weights, n_vec, n_heads, G)
    cb = _cb(codebooks, n_heads, D, c, b)
    out = np.empty_like(cb)
    codes = np.empty((n_vec, n_heads, G), dtype=np.int32)
    obj = np.empty((n_heads, G), dtype=np.float64)
    _load().oracle_lloyd_step(_p(xb), _p(w), _p(cb), n_vec, n_heads, D, c, b, _p(out), _p(codes), _p(obj))
    return out, codes, obj
