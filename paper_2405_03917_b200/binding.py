"""ctypes binding of `libcq.so`: argument marshalling only, same names as the C ABI.

Every function takes torch tensors (device tensors for device pointers, CPU tensors for
the `_host` arguments), checks dtype / contiguity / device, and forwards raw pointers and
sizes.  A non-zero cq_status raises CQError.  Work is enqueued on torch's current stream.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libcq.so")

# Every symbol include/cq.h declares.
EXPORTS = ["cq_layout_version", "cq_status_string", "cq_codes_bytes", "cq_encode", "cq_encode_variant", "cq_encode_kv",
           "cq_codes_to_rowmajor", "cq_codes_from_rowmajor", "cq_decode_attn_workspace_bytes", "cq_decode_attn",
           "cq_decode_attn_variant", "cq_decode_attn_rope", "cq_decode_attn_rope_variant", "cq_prefill_attn", "cq_prefill_attn_variant", "cq_decode_attn_static", "cq_decode_step_workspace_bytes", "cq_decode_step_launches", "cq_decode_step", "cq_decode_step_host_workspace_bytes",
           "cq_decode_step_host", "cq_learn_workspace_bytes", "cq_kmeanspp_init", "cq_lloyd_step", "cq_learn_centroids"]


class CQError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {cq_status_string(status)} ({status})")


_lib = None


def library_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2405_03917_b200.build` "
                              "(needs nvcc); this package has no CPU or PyTorch fallback")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i64, i32, f32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.cq_layout_version.restype = i32
        L.cq_status_string.restype = ctypes.c_char_p
        L.cq_status_string.argtypes = [i32]
        L.cq_codes_bytes.restype = sz
        L.cq_codes_bytes.argtypes = [i64, i64, i32, i32, i32, i32]
        L.cq_encode.restype = i32
        L.cq_encode.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, i32, i32, i32, vp, vp]
        L.cq_encode_variant.restype = i32
        L.cq_encode_variant.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, i32, i32, i32, vp, i32, vp]
        for f in (L.cq_codes_to_rowmajor, L.cq_codes_from_rowmajor):
            f.restype = i32
            f.argtypes = [vp, i64, i64, i32, i32, i32, i32, vp, vp]
        L.cq_decode_attn_workspace_bytes.restype = sz
        L.cq_decode_attn_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i64]
        L.cq_decode_attn.restype = i32
        L.cq_decode_attn.argtypes = [vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i64, vp, vp, sz, vp]
        for f in (L.cq_prefill_attn, L.cq_prefill_attn_variant):
            f.restype = i32
        L.cq_prefill_attn.argtypes = [vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i32, i64, vp, vp]
        L.cq_prefill_attn_variant.argtypes = [vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i32, i64, vp, i32, vp]
        L.cq_decode_attn_variant.restype = i32
        L.cq_decode_attn_variant.argtypes = [vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i64, vp, vp,
                                             sz, i32, vp]
        L.cq_encode_kv.restype = i32
        L.cq_encode_kv.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp]
        L.cq_decode_attn_rope.restype = i32
        L.cq_decode_attn_rope.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, i32, i32, i32, i32, i32, i64,
                                          vp, vp, sz, vp]
        L.cq_decode_attn_rope_variant.restype = i32
        L.cq_decode_attn_rope_variant.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, f32, i32, i32, i32, i32, i32, i32, i64,
                                          vp, vp, sz, i32, vp]
        L.cq_decode_attn_static.restype = i32
        L.cq_decode_attn_static.argtypes = [vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i64, vp, vp]
        L.cq_learn_workspace_bytes.restype = sz
        L.cq_learn_workspace_bytes.argtypes = [i64, i32, i32, i32, i32]
        L.cq_kmeanspp_init.restype = i32
        L.cq_kmeanspp_init.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, sz, vp]
        L.cq_lloyd_step.restype = i32
        L.cq_lloyd_step.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.cq_learn_centroids.restype = i32
        L.cq_learn_centroids.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.cq_decode_step_workspace_bytes.restype = sz
        L.cq_decode_step_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i64]
        L.cq_decode_step_launches.restype = i32
        L.cq_decode_step_launches.argtypes = [i32, i32, i32, i32, i32, i32, i64]
        L.cq_decode_step.restype = i32
        L.cq_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i64, vp, vp, sz, vp]
        L.cq_decode_step_host_workspace_bytes.restype = sz
        L.cq_decode_step_host_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i64]
        L.cq_decode_step_host.restype = i32
        L.cq_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32, i64,
                                          vp, vp, sz, vp]
        _lib = L
    return _lib


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name}: CUDA tensor expected")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: contiguous {dtype} tensor expected, got {t.dtype}")
    return t.data_ptr()


def _host(t: torch.Tensor, dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name}: CPU tensor expected")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: contiguous {dtype} tensor expected, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str) -> None:
    if status != 0:
        raise CQError(status, where)


def cq_layout_version() -> int:
    return int(lib().cq_layout_version())


def cq_status_string(status: int) -> str:
    return lib().cq_status_string(int(status)).decode()


def cq_codes_bytes(n_seq: int, max_tokens: int, n_heads: int, head_dim: int, c: int, b: int) -> int:
    return int(lib().cq_codes_bytes(n_seq, max_tokens, n_heads, head_dim, c, b))


def cq_encode(x: torch.Tensor, codebooks: torch.Tensor, c: int, b: int, codes_out: torch.Tensor, max_tokens: int,
              token_offset: int = 0, seq_offsets: Optional[torch.Tensor] = None, variant: int = 0) -> torch.Tensor:
    """x fp16 (n_seq, n_tokens, n_heads, head_dim); codebooks fp32 (n_heads, G, 2^b, c);
    codes_out uint8 buffer of cq_codes_bytes(...) bytes, updated in place and returned."""
    n_seq, n_tokens, n_heads, head_dim = x.shape
    if tuple(codebooks.shape) != (n_heads, head_dim // max(c, 1), 1 << b, c):
        raise ValueError(f"codebooks shape {tuple(codebooks.shape)} does not match heads/groups/centroids")
    need = cq_codes_bytes(n_seq, max_tokens, n_heads, head_dim, c, b)
    if need and codes_out.numel() < need:
        raise ValueError(f"codes_out holds {codes_out.numel()} bytes, {need} needed")
    so = None if seq_offsets is None else _dev(seq_offsets, torch.int32, "seq_offsets")
    if seq_offsets is not None and seq_offsets.numel() != n_seq:
        raise ValueError("seq_offsets must have n_seq entries")
    st = lib().cq_encode_variant(_dev(x, torch.float16, "x"), _dev(codebooks, torch.float32, "codebooks"), so,
                                 n_seq, n_tokens, token_offset, max_tokens, n_heads, head_dim, c, b,
                                 _dev(codes_out, torch.uint8, "codes_out"), variant, _stream())
    _check(st, "cq_encode")
    return codes_out


def cq_encode_kv(k: torch.Tensor, v: torch.Tensor, k_cb: torch.Tensor, v_cb: torch.Tensor, c: int, b: int,
                 k_codes_out: torch.Tensor, v_codes_out: torch.Tensor, max_tokens: int, token_offset: int = 0,
                 seq_offsets: Optional[torch.Tensor] = None) -> None:
    """cq_encode of the key and the value embeddings of the same tokens; k, v fp16 (n_seq, n_tokens, n_heads, head_dim)."""
    n_seq, n_tokens, n_heads, head_dim = k.shape
    if tuple(v.shape) != tuple(k.shape):
        raise ValueError("k and v must have the same shape")
    so = None if seq_offsets is None else _dev(seq_offsets, torch.int32, "seq_offsets")
    st = lib().cq_encode_kv(_dev(k, torch.float16, "k"), _dev(v, torch.float16, "v"), _dev(k_cb, torch.float32, "k_cb"),
                            _dev(v_cb, torch.float32, "v_cb"), so, n_seq, n_tokens, token_offset, max_tokens, n_heads,
                            head_dim, c, b, _dev(k_codes_out, torch.uint8, "k_codes_out"),
                            _dev(v_codes_out, torch.uint8, "v_codes_out"), _stream())
    _check(st, "cq_encode_kv")


def cq_codes_to_rowmajor(codes: torch.Tensor, n_seq: int, max_tokens: int, n_heads: int, head_dim: int, c: int,
                         b: int) -> torch.Tensor:
    # one byte per code for b <= 8, else two (returned as int16 holding the unsigned 16-bit pattern)
    out = torch.empty(n_seq, max_tokens, n_heads, head_dim // c, dtype=torch.uint8 if b <= 8 else torch.int16,
                      device=codes.device)
    st = lib().cq_codes_to_rowmajor(_dev(codes, torch.uint8, "codes"), n_seq, max_tokens, n_heads, head_dim, c, b,
                                    out.data_ptr(), _stream())
    _check(st, "cq_codes_to_rowmajor")
    return out


def cq_codes_from_rowmajor(rowmajor: torch.Tensor, head_dim: int, c: int, b: int) -> torch.Tensor:
    n_seq, max_tokens, n_heads, G = rowmajor.shape
    if G * c != head_dim:
        raise ValueError("last dimension must be head_dim / c")
    out = torch.empty(cq_codes_bytes(n_seq, max_tokens, n_heads, head_dim, c, b), dtype=torch.uint8,
                      device=rowmajor.device)
    st = lib().cq_codes_from_rowmajor(_dev(rowmajor, torch.uint8 if b <= 8 else torch.int16, "rowmajor"), n_seq, max_tokens, n_heads, head_dim,
                                      c, b, out.data_ptr(), _stream())
    _check(st, "cq_codes_from_rowmajor")
    return out


def cq_decode_attn_workspace_bytes(n_seq: int, n_q_heads: int, n_kv_heads: int, head_dim: int, c: int, b: int,
                                   max_tokens: int) -> int:
    return int(lib().cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens))


def cq_decode_attn(q: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor, k_cb: torch.Tensor,
                   v_cb: torch.Tensor, seq_lens: torch.Tensor, scale: float, c: int, b: int, max_tokens: int,
                   out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   variant: int = 0) -> torch.Tensor:
    """q fp16 (n_seq, Hq, head_dim); codes in the library layout; codebooks fp32
    (Hkv, G, 2^b, c); seq_lens int32 (n_seq,).  Returns out fp32 (n_seq, Hq, head_dim)."""
    n_seq, n_q_heads, head_dim = q.shape
    n_kv_heads = k_cb.shape[0]
    for nm, cb in (("k_cb", k_cb), ("v_cb", v_cb)):
        if tuple(cb.shape) != (n_kv_heads, head_dim // max(c, 1), 1 << b, c):
            raise ValueError(f"{nm} shape {tuple(cb.shape)} does not match heads/groups/centroids")
    need_codes = cq_codes_bytes(n_seq, max_tokens, n_kv_heads, head_dim, c, b)
    if need_codes and (k_codes.numel() < need_codes or v_codes.numel() < need_codes):
        raise ValueError(f"code buffers must hold {need_codes} bytes")
    if seq_lens.numel() != n_seq:
        raise ValueError("seq_lens must have n_seq entries")
    if out is None:
        out = torch.empty(n_seq, n_q_heads, head_dim, dtype=torch.float32, device=q.device)
    if workspace is None:
        nbytes = cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens)
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    st = lib().cq_decode_attn_variant(_dev(q, torch.float16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                      _dev(v_codes, torch.uint8, "v_codes"), _dev(k_cb, torch.float32, "k_cb"),
                                      _dev(v_cb, torch.float32, "v_cb"), _dev(seq_lens, torch.int32, "seq_lens"),
                                      float(scale), n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens,
                                      _dev(out, torch.float32, "out"), _dev(workspace, torch.uint8, "workspace"),
                                      workspace.numel(), variant, _stream())
    _check(st, "cq_decode_attn")
    return out


def cq_prefill_attn(q: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor, k_cb: torch.Tensor,
                    v_cb: torch.Tensor, seq_lens: torch.Tensor, scale: float, c: int, b: int, max_tokens: int,
                    out: Optional[torch.Tensor] = None, variant: int = 0) -> torch.Tensor:
    """Causal attention of the n_q newest cached tokens.  q fp16 (n_seq, n_q, Hq, head_dim); seq_lens counts
    the cached tokens including the new ones.  Returns out fp32 (n_seq, n_q, Hq, head_dim)."""
    n_seq, n_q, n_q_heads, head_dim = q.shape
    n_kv_heads = k_cb.shape[0]
    for nm, cb in (("k_cb", k_cb), ("v_cb", v_cb)):
        if tuple(cb.shape) != (n_kv_heads, head_dim // max(c, 1), 1 << b, c):
            raise ValueError(f"{nm} shape {tuple(cb.shape)} does not match heads/groups/centroids")
    need_codes = cq_codes_bytes(n_seq, max_tokens, n_kv_heads, head_dim, c, b)
    if need_codes and (k_codes.numel() < need_codes or v_codes.numel() < need_codes):
        raise ValueError(f"code buffers must hold {need_codes} bytes")
    if seq_lens.numel() != n_seq:
        raise ValueError("seq_lens must have n_seq entries")
    if out is None:
        out = torch.empty(n_seq, n_q, n_q_heads, head_dim, dtype=torch.float32, device=q.device)
    st = lib().cq_prefill_attn_variant(_dev(q, torch.float16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                       _dev(v_codes, torch.uint8, "v_codes"), _dev(k_cb, torch.float32, "k_cb"),
                                       _dev(v_cb, torch.float32, "v_cb"), _dev(seq_lens, torch.int32, "seq_lens"),
                                       float(scale), n_seq, n_q, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens,
                                       _dev(out, torch.float32, "out"), variant, _stream())
    _check(st, "cq_prefill_attn")
    return out


STATIC_WORKSPACE_BYTES = 4 << 20      # CQ_STATIC_WORKSPACE_BYTES of include/cq.h


ROPE_HALF, ROPE_INTERLEAVED = 0, 1


def cq_decode_attn_rope(q: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor, k_cb: torch.Tensor,
                        v_cb: torch.Tensor, seq_lens: torch.Tensor, rope_cos: torch.Tensor, rope_sin: torch.Tensor,
                        scale: float, c: int, b: int, max_tokens: int, pairing: int = ROPE_HALF,
                        out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                        variant: int = 0) -> torch.Tensor:
    """cq_decode_attn for key codes taken before RoPE: rope_cos / rope_sin fp32 (max_tokens, head_dim / 2).
    variant 0 = automatic, 1 = generic kernel, 2 = tuned kernel."""
    n_seq, n_q_heads, head_dim = q.shape
    n_kv_heads = k_cb.shape[0]
    for nm, t in (("rope_cos", rope_cos), ("rope_sin", rope_sin)):
        if tuple(t.shape) != (max_tokens, head_dim // 2):
            raise ValueError(f"{nm} shape {tuple(t.shape)}, expected {(max_tokens, head_dim // 2)}")
    need_codes = cq_codes_bytes(n_seq, max_tokens, n_kv_heads, head_dim, c, b)
    if need_codes and (k_codes.numel() < need_codes or v_codes.numel() < need_codes):
        raise ValueError(f"code buffers must hold {need_codes} bytes")
    if out is None:
        out = torch.empty(n_seq, n_q_heads, head_dim, dtype=torch.float32, device=q.device)
    if workspace is None:
        nbytes = cq_decode_attn_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens)
        workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
    st = lib().cq_decode_attn_rope_variant(_dev(q, torch.float16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                   _dev(v_codes, torch.uint8, "v_codes"), _dev(k_cb, torch.float32, "k_cb"),
                                   _dev(v_cb, torch.float32, "v_cb"), _dev(seq_lens, torch.int32, "seq_lens"),
                                   _dev(rope_cos, torch.float32, "rope_cos"), _dev(rope_sin, torch.float32, "rope_sin"),
                                   int(pairing), float(scale), n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens,
                                   _dev(out, torch.float32, "out"), _dev(workspace, torch.uint8, "workspace"),
                                   workspace.numel(), int(variant), _stream())
    _check(st, "cq_decode_attn_rope")
    return out


def cq_decode_attn_static(q: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor, k_cb: torch.Tensor,
                          v_cb: torch.Tensor, seq_lens: torch.Tensor, scale: float, c: int, b: int, max_tokens: int,
                          out: torch.Tensor) -> torch.Tensor:
    """cq_decode_attn without a workspace: the partials go to the array built into the library
    (shapes that need more than STATIC_WORKSPACE_BYTES raise CQError with CQ_ERR_WORKSPACE).
    This wrapper allocates nothing either: `out` is the caller's.  Calls that overlap on the
    GPU share the array and must be ordered by the caller."""
    n_seq, n_q_heads, head_dim = q.shape
    n_kv_heads = k_cb.shape[0]
    # the same shape checks as cq_decode_attn (they allocate nothing)
    for nm, cb in (("k_cb", k_cb), ("v_cb", v_cb)):
        if tuple(cb.shape) != (n_kv_heads, head_dim // max(c, 1), 1 << b, c):
            raise ValueError(f"{nm} shape {tuple(cb.shape)} does not match heads/groups/centroids")
    need_codes = cq_codes_bytes(n_seq, max_tokens, n_kv_heads, head_dim, c, b)
    if need_codes and (k_codes.numel() < need_codes or v_codes.numel() < need_codes):
        raise ValueError(f"code buffers must hold {need_codes} bytes")
    if seq_lens.numel() != n_seq:
        raise ValueError("seq_lens must have n_seq entries")
    st = lib().cq_decode_attn_static(_dev(q, torch.float16, "q"), _dev(k_codes, torch.uint8, "k_codes"),
                                     _dev(v_codes, torch.uint8, "v_codes"), _dev(k_cb, torch.float32, "k_cb"),
                                     _dev(v_cb, torch.float32, "v_cb"), _dev(seq_lens, torch.int32, "seq_lens"),
                                     float(scale), n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens,
                                     _dev(out, torch.float32, "out"), _stream())
    _check(st, "cq_decode_attn_static")
    return out


def cq_decode_step_workspace_bytes(n_seq: int, n_q_heads: int, n_kv_heads: int, head_dim: int, c: int, b: int,
                                   max_tokens: int) -> int:
    return int(lib().cq_decode_step_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens))


def cq_decode_step_launches(n_seq: int, n_q_heads: int, n_kv_heads: int, head_dim: int, c: int, b: int, max_tokens: int) -> int:
    """Kernel launches of one cq_decode_step call on this shape."""
    return int(lib().cq_decode_step_launches(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens))


def cq_decode_step(q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, seq_lens: torch.Tensor,
                   k_codes: torch.Tensor, v_codes: torch.Tensor, k_cb: torch.Tensor, v_cb: torch.Tensor, scale: float,
                   c: int, b: int, max_tokens: int, out: Optional[torch.Tensor] = None,
                   workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One decode step on device buffers: q fp16 (n_seq, n_q_heads, D), k_new / v_new fp16 (n_seq, n_kv_heads, D),
    seq_lens int32 (n_seq,) = tokens cached before the step.  The caches take the new token's codes; returns the
    attention output fp32 (n_seq, n_q_heads, D) over seq_lens + 1 tokens."""
    n_seq, n_q_heads, head_dim = q.shape
    n_kv_heads = k_cb.shape[0]
    if tuple(k_new.shape) != (n_seq, n_kv_heads, head_dim) or tuple(v_new.shape) != (n_seq, n_kv_heads, head_dim):
        raise ValueError("k_new and v_new must be (n_seq, n_kv_heads, head_dim)")
    if seq_lens.numel() != n_seq:
        raise ValueError("seq_lens must have n_seq entries")
    need_codes = cq_codes_bytes(n_seq, max_tokens, n_kv_heads, head_dim, c, b)
    if need_codes and (k_codes.numel() < need_codes or v_codes.numel() < need_codes):
        raise ValueError(f"code buffers hold {k_codes.numel()} / {v_codes.numel()} bytes, {need_codes} needed")
    need = cq_decode_step_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty(n_seq, n_q_heads, head_dim, dtype=torch.float32, device=q.device)
    st = lib().cq_decode_step(_dev(q, torch.float16, "q"), _dev(k_new, torch.float16, "k_new"), _dev(v_new, torch.float16, "v_new"),
                              _dev(seq_lens, torch.int32, "seq_lens"), _dev(k_codes, torch.uint8, "k_codes"),
                              _dev(v_codes, torch.uint8, "v_codes"), _dev(k_cb, torch.float32, "k_cb"),
                              _dev(v_cb, torch.float32, "v_cb"), float(scale), n_seq, n_q_heads, n_kv_heads, head_dim, c, b,
                              max_tokens, _dev(out, torch.float32, "out"), _dev(workspace, torch.uint8, "workspace"),
                              workspace.numel(), _stream())
    _check(st, "cq_decode_step")
    return out


def cq_decode_step_host_workspace_bytes(n_seq: int, n_q_heads: int, n_kv_heads: int, head_dim: int, c: int, b: int,
                                        max_tokens: int) -> int:
    return int(lib().cq_decode_step_host_workspace_bytes(n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens))


def cq_decode_step_host(q_host: torch.Tensor, k_new_host: torch.Tensor, v_new_host: torch.Tensor,
                        seq_lens_host: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor,
                        k_cb: torch.Tensor, v_cb: torch.Tensor, scale: float, c: int, b: int, max_tokens: int,
                        out_host: torch.Tensor, workspace: torch.Tensor) -> torch.Tensor:
    """One decode step from host buffers: H2D copies, append-encode, attention, D2H copy, stream sync."""
    n_seq, n_q_heads, head_dim = q_host.shape
    n_kv_heads = k_cb.shape[0]
    st = lib().cq_decode_step_host(_host(q_host, torch.float16, "q_host"), _host(k_new_host, torch.float16, "k_new_host"),
                                   _host(v_new_host, torch.float16, "v_new_host"),
                                   _host(seq_lens_host, torch.int32, "seq_lens_host"),
                                   _dev(k_codes, torch.uint8, "k_codes"), _dev(v_codes, torch.uint8, "v_codes"),
                                   _dev(k_cb, torch.float32, "k_cb"), _dev(v_cb, torch.float32, "v_cb"), float(scale),
                                   n_seq, n_q_heads, n_kv_heads, head_dim, c, b, max_tokens,
                                   _host(out_host, torch.float32, "out_host"),
                                   _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream())
    _check(st, "cq_decode_step_host")
    return out_host


# ------------------------------------------------------------------------------ centroid learning

def cq_learn_workspace_bytes(n_vec: int, n_heads: int, head_dim: int, c: int, b: int) -> int:
    return int(lib().cq_learn_workspace_bytes(n_vec, n_heads, head_dim, c, b))


def _learn_common(x, weights, c, b):
    n_vec, n_heads, head_dim = x.shape
    G = head_dim // max(c, 1)
    if weights is not None and tuple(weights.shape) != (n_vec, n_heads, G):
        raise ValueError(f"weights shape {tuple(weights.shape)}, expected {(n_vec, n_heads, G)}")
    wp = None if weights is None else _dev(weights, torch.float32, "weights")
    ws = torch.empty(max(256, cq_learn_workspace_bytes(n_vec, n_heads, head_dim, c, b)), dtype=torch.uint8, device=x.device)
    return n_vec, n_heads, head_dim, G, wp, ws


def cq_kmeanspp_init(x: torch.Tensor, weights: Optional[torch.Tensor], uniforms: torch.Tensor, c: int, b: int) -> torch.Tensor:
    """x fp16 (n_vec, n_heads, head_dim); weights fp32 (n_vec, n_heads, G) or None; uniforms fp64
    (n_heads, G, 2^b).  Returns the initial codebooks fp32 (n_heads, G, 2^b, c)."""
    n_vec, n_heads, head_dim, G, wp, ws = _learn_common(x, weights, c, b)
    if tuple(uniforms.shape) != (n_heads, G, 1 << b):
        raise ValueError("uniforms must be (n_heads, G, 2^b)")
    out = torch.empty(n_heads, G, 1 << b, c, dtype=torch.float32, device=x.device)
    st = lib().cq_kmeanspp_init(_dev(x, torch.float16, "x"), wp, _dev(uniforms, torch.float64, "uniforms"), n_vec, n_heads,
                                head_dim, c, b, out.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "cq_kmeanspp_init")
    return out


def cq_lloyd_step(x: torch.Tensor, weights: Optional[torch.Tensor], codebooks: torch.Tensor, c: int, b: int):
    """One k-means iteration.  Returns (new codebooks, objective fp64 (n_heads, G) of the assignment)."""
    n_vec, n_heads, head_dim, G, wp, ws = _learn_common(x, weights, c, b)
    out = torch.empty_like(codebooks)
    obj = torch.empty(n_heads, G, dtype=torch.float64, device=x.device)
    st = lib().cq_lloyd_step(_dev(x, torch.float16, "x"), wp, _dev(codebooks, torch.float32, "codebooks"), n_vec, n_heads,
                             head_dim, c, b, out.data_ptr(), obj.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "cq_lloyd_step")
    return out, obj


def cq_learn_centroids(x: torch.Tensor, weights: Optional[torch.Tensor], uniforms: torch.Tensor, c: int, b: int,
                       n_iters: int):
    """k-means++ initialisation and n_iters k-means iterations.  Returns (codebooks, objective of the
    last assignment)."""
    n_vec, n_heads, head_dim, G, wp, ws = _learn_common(x, weights, c, b)
    out = torch.empty(n_heads, G, 1 << b, c, dtype=torch.float32, device=x.device)
    obj = torch.zeros(n_heads, G, dtype=torch.float64, device=x.device)
    st = lib().cq_learn_centroids(_dev(x, torch.float16, "x"), wp, _dev(uniforms, torch.float64, "uniforms"), n_vec,
                                  n_heads, head_dim, c, b, n_iters, out.data_ptr(), obj.data_ptr(), ws.data_ptr(),
                                  ws.numel(), _stream())
    _check(st, "cq_learn_centroids")
    return out, obj
