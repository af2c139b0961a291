"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, sizes follow the documented layout, and invalid
arguments are rejected before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import build as cq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    cq_build.build()
    return cq.lib()


def header_functions():
    text = open(os.path.join(ROOT, "include", "cq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cq_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = header_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in include/cq.h but not exported"
    assert sorted(cq.EXPORTS) == names


def test_layout_version_and_status_strings(L):
    assert cq.cq_layout_version() == 1
    assert cq.cq_status_string(0) == "CQ_OK"
    for st in range(-6, 0):
        assert cq.cq_status_string(st).startswith("CQ_ERR_")
    assert "unknown" in cq.cq_status_string(17)


def test_code_buffer_sizes():
    # one byte per (token, head, group), capacity rounded up to 16-token blocks
    assert cq.cq_codes_bytes(1, 1024, 1, 128, 8, 8) == 1024 * 16
    assert cq.cq_codes_bytes(16, 4096, 32, 128, 4, 8) == 16 * 4096 * 32 * 32          # 64 MiB (config 1)
    assert cq.cq_codes_bytes(64, 16384, 8, 128, 8, 8) == 64 * 16384 * 8 * 16          # 128 MiB (config 2)
    assert cq.cq_codes_bytes(8, 8192, 32, 128, 2, 8) == 8 * 8192 * 32 * 64            # 128 MiB (config 3)
    assert cq.cq_codes_bytes(2, 17, 3, 64, 4, 5) == 2 * 3 * 2 * 16 * 16               # 17 tokens -> 2 blocks
    # invalid shapes give 0
    assert cq.cq_codes_bytes(1, 16, 1, 128, 3, 8) == 0      # c does not divide head_dim
    # codes wider than a byte: 16 low bytes + 2 (b - 8) bytes of upper bits per (block, group);
    # CQ-8c10b is 10 bits per 8 channels = 1.25 bits per channel (Table 1)
    assert cq.cq_codes_bytes(1, 16, 1, 128, 8, 10) == 16 * 20
    assert cq.cq_codes_bytes(1, 16, 1, 128, 8, 10) * 8 / (16 * 128) == 1.25
    assert cq.cq_codes_bytes(2, 17, 3, 64, 8, 12) == 2 * 3 * 2 * 8 * 24
    assert cq.cq_codes_bytes(1, 16, 1, 8, 8, 9) == 32       # 18 bytes, rounded up to a multiple of 16
    assert cq.cq_codes_bytes(1, 16, 1, 128, 8, 11) == 0     # widths whose upper bits would straddle bytes
    assert cq.cq_codes_bytes(1, 16, 1, 128, 8, 17) == 0
    assert cq.cq_codes_bytes(0, 16, 1, 128, 8, 8) == 0
    assert cq.cq_codes_bytes(1, 16, 1, 512, 8, 8) == 0      # head_dim > 256


def test_workspace_sizes_are_positive_and_reject_bad_shapes():
    assert cq.cq_decode_attn_workspace_bytes(64, 32, 8, 128, 8, 8, 16384) > 0
    assert cq.cq_decode_attn_workspace_bytes(64, 32, 5, 128, 8, 8, 16384) == 0   # Hq % Hkv
    assert cq.cq_decode_step_host_workspace_bytes(4, 8, 2, 128, 8, 8, 100) > \
        cq.cq_decode_attn_workspace_bytes(4, 8, 2, 128, 8, 8, 100)


def test_argument_validation_happens_on_the_host(L):
    # Fake, suitably aligned non-NULL addresses: every call below must fail validation
    # before touching them (nothing is launched, so no GPU is needed).
    p = 0x10000
    enc = lambda **kw: L.cq_encode(*[kw.get(k, d) for k, d in [
        ("x", p), ("cb", p), ("so", None), ("n_seq", 1), ("n_tok", 4), ("off", 0), ("cap", 16),
        ("heads", 1), ("D", 128), ("c", 8), ("b", 8), ("out", p), ("stream", None)]])
    assert enc(x=None) == -1
    assert enc(out=None) == -1
    assert enc(c=3) == -2
    assert enc(n_seq=0) == -2
    assert enc(n_tok=17) == -2                 # past capacity
    assert enc(off=-1) == -2
    assert enc(b=0) == -3
    assert enc(b=11) == -3                     # a width whose upper bits would straddle bytes
    assert enc(D=512, c=8) == -3
    assert enc(x=p + 2) == -4
    assert enc(n_tok=0) == 0                   # nothing to do, nothing launched

    dec = lambda **kw: L.cq_decode_attn(*[kw.get(k, d) for k, d in [
        ("q", p), ("kc", p), ("vc", p), ("kcb", p), ("vcb", p), ("sl", p), ("scale", ctypes.c_float(0.1)),
        ("n_seq", 2), ("hq", 4), ("hkv", 2), ("D", 128), ("c", 8), ("b", 8), ("cap", 64), ("out", p),
        ("ws", p), ("ws_bytes", 1 << 30), ("stream", None)]])
    assert dec(q=None) == -1
    assert dec(ws=None) == -1
    assert dec(hkv=3) == -2
    assert dec(c=5) == -2
    assert dec(b=12) == -3
    assert dec(kc=p + 8) == -4
    assert dec(ws_bytes=16) == -5
    conv = L.cq_codes_to_rowmajor(None, 1, 16, 1, 128, 8, 8, p, None)
    assert conv == -1
    # cq_encode_kv: the two code buffers must differ; the same checks as cq_encode otherwise
    kv = lambda **kw: L.cq_encode_kv(*[kw.get(k, d) for k, d in [
        ("k", p), ("v", p), ("kcb", p), ("vcb", p), ("so", None), ("n_seq", 1), ("n_tok", 4), ("off", 0), ("cap", 16),
        ("heads", 1), ("D", 128), ("c", 8), ("b", 8), ("ko", p), ("vo", p + 4096), ("stream", None)]])
    assert kv(v=None) == -1
    assert kv(vo=p) == -2
    assert kv(n_tok=17) == -2
    assert kv(b=11) == -3
    assert kv(ko=p + 4) == -4
    # cq_decode_attn_rope: tables are required, the pairing is 0 or 1, a pair must lie in whole groups
    rope = lambda **kw: L.cq_decode_attn_rope(*[kw.get(k, d) for k, d in [
        ("q", p), ("kc", p), ("vc", p), ("kcb", p), ("vcb", p), ("sl", p), ("cos", p), ("sin", p), ("pairing", 0),
        ("scale", ctypes.c_float(0.1)), ("n_seq", 2), ("hq", 4), ("hkv", 2), ("D", 128), ("c", 8), ("b", 8), ("cap", 64),
        ("out", p), ("ws", p), ("ws_bytes", 1 << 30), ("stream", None)]])
    assert rope(cos=None) == -1
    assert rope(pairing=2) == -2
    assert rope(c=128, b=2) == -3              # one group: channel i + 64 cannot be in another group's code
    assert rope(c=1, b=2, pairing=1) == -3     # an interleaved pair would span two groups
    assert rope(cos=p + 2) == -4
    assert rope(ws_bytes=16) == -5


def test_new_entry_points_validate_on_the_host(L):
    p = 0x10000
    f32 = ctypes.c_float
    # cq_decode_step: null pointers, shapes, alignment of the new key / value, aliasing caches, workspace size
    step = lambda **kw: L.cq_decode_step(*[kw.get(k, d) for k, d in [
        ("q", p), ("k", p), ("v", p), ("sl", p), ("kc", p), ("vc", p + 4096), ("kcb", p), ("vcb", p), ("scale", f32(0.1)),
        ("n_seq", 2), ("hq", 8), ("hkv", 2), ("D", 128), ("c", 8), ("b", 8), ("cap", 64), ("out", p), ("ws", p),
        ("ws_bytes", 1 << 30), ("stream", None)]])
    assert step(k=None) == -1
    assert step(sl=None) == -1
    assert step(hkv=3) == -2
    assert step(vc=p) == -2                    # the two caches must be different buffers
    assert step(b=11) == -3
    assert step(k=p + 2) == -4
    assert step(ws_bytes=64) == -5
    # launches of a step: the attention kernel appends and writes the output (1), plus a merge for split contexts (2),
    # or lengths + append + attention + merge (4) where no kernel appends; 0 for a shape the library refuses
    assert cq.cq_decode_step_launches(64, 32, 8, 128, 8, 8, 16384) in (1, 2)
    assert cq.cq_decode_step_launches(16, 32, 32, 128, 4, 8, 4096) in (1, 2)
    assert cq.cq_decode_step_launches(2, 8, 2, 128, 8, 8, 1 << 20) == 2          # few long contexts: split, so a merge follows
    assert cq.cq_decode_step_launches(16, 32, 32, 128, 8, 10, 8192) == 4         # CQ-8c10b: no appending kernel
    assert cq.cq_decode_step_launches(2, 4, 2, 64, 4, 5, 100) == 4
    assert cq.cq_decode_step_launches(2, 4, 3, 64, 4, 5, 100) == 0
    assert cq.cq_decode_step_workspace_bytes(4, 8, 2, 128, 8, 8, 100) > cq.cq_decode_attn_workspace_bytes(4, 8, 2, 128, 8, 8, 100)

    # cq_prefill_attn: more queries than the cache holds, bad variant, null pointers
    pre = lambda **kw: L.cq_prefill_attn_variant(*[kw.get(k, d) for k, d in [
        ("q", p), ("kc", p), ("vc", p), ("kcb", p), ("vcb", p), ("sl", p), ("scale", f32(0.1)), ("n_seq", 1), ("n_q", 4),
        ("hq", 4), ("hkv", 2), ("D", 128), ("c", 8), ("b", 8), ("cap", 64), ("out", p), ("variant", 0), ("stream", None)]])
    assert pre(q=None) == -1
    assert pre(n_q=65) == -2
    assert pre(variant=7) == -2
    assert pre(hkv=3) == -2
    assert pre(b=10, variant=2) == -3          # the tensor-core kernel takes byte codes only

    # cq_decode_attn_rope_variant: pairing, groups that a pair would split, the tuned kernel's shapes
    rope = lambda **kw: L.cq_decode_attn_rope_variant(*[kw.get(k, d) for k, d in [
        ("q", p), ("kc", p), ("vc", p), ("kcb", p), ("vcb", p), ("sl", p), ("cos", p), ("sin", p), ("pairing", 0),
        ("scale", f32(0.1)), ("n_seq", 1), ("hq", 4), ("hkv", 2), ("D", 128), ("c", 8), ("b", 8), ("cap", 64),
        ("out", p), ("ws", p), ("ws_bytes", 1 << 30), ("variant", 0), ("stream", None)]])
    assert rope(cos=None) == -1
    assert rope(pairing=2) == -2
    assert rope(variant=3) == -2
    assert rope(pairing=1, variant=2) == -3    # the tuned kernel pairs (i, i + 64) only
    assert rope(c=2, variant=2) == -3
    assert rope(cos=p + 4, variant=2) == -3    # tables must be 8-byte aligned for it
    assert rope(cos=p + 2) == -4

    # cq_encode_variant 4: the tensor-memory kernel takes byte codes of head_dim 128 only
    encv = lambda **kw: L.cq_encode_variant(*[kw.get(k, d) for k, d in [
        ("x", p), ("cb", p), ("so", None), ("n_seq", 1), ("n_tok", 4), ("off", 0), ("cap", 16),
        ("heads", 1), ("D", 128), ("c", 8), ("b", 8), ("out", p), ("variant", 4), ("stream", None)]])
    assert encv(b=10) == -3
    assert encv(D=64) == -3
    assert encv(variant=5) == -2
