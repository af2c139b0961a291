"""cq_decode_attn_static: decode attention for callers that cannot allocate device memory.

Some users of this library run where a workspace cannot be had: the serving process gave
all of HBM to its KV-cache pool when it started, or the library sits behind a plug-in
interface that passes only input and output pointers.  For them the C ABI has one entry
point whose split-K partials live in an array built into the library.  This test drives it
through the C ABI twice in a row, with different inputs, and compares each result with
what the ordinary entry point (caller-owned workspace) returns for the same inputs, under
the attention tolerance the other tests use.  The second call finds the first call's
partials still in the array; they must not leak into its result.

The file name sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def build_case(config, n_seq, n_q, n_kv, cap, c=8, b=8):
    w = H.small_workload("static", config, c, b, n_seq, n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, n_seq, cap)
    xv = synth.layer_activations(w, 0, True, n_seq, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(config, 0, n_seq, n_q)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    kb = cq.cq_codes_from_rowmajor(torch.from_numpy(kc_rm.astype(np.uint8)).to(DEV), 128, c, b)
    vb = cq.cq_codes_from_rowmajor(torch.from_numpy(vc_rm.astype(np.uint8)).to(DEV), 128, c, b)
    return dict(q=q.to(DEV), kb=kb, vb=vb, kcb=kcb.to(DEV), vcb=vcb.to(DEV), c=c, b=b, cap=cap,
                host=(q, kc_rm, vc_rm, kcb, vcb))


def run_both(case, lens):
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    scale = 128 ** -0.5
    ref = cq.cq_decode_attn(case["q"], case["kb"], case["vb"], case["kcb"], case["vcb"], sl, scale,
                            case["c"], case["b"], case["cap"])
    out = torch.full_like(ref, float("nan"))
    cq.cq_decode_attn_static(case["q"], case["kb"], case["vb"], case["kcb"], case["vcb"], sl, scale,
                             case["c"], case["b"], case["cap"], out)
    torch.cuda.synchronize()
    return out.cpu().numpy(), ref.cpu().numpy()


def test_static_workspace_matches_caller_workspace_on_two_calls_in_a_row():
    # first call: GQA, several context chunks, ragged lengths and an empty sequence
    a = build_case(881, 3, 4, 1, 5000)
    lens_a = [5000, 0, 2049]
    out, ref = run_both(a, lens_a)
    H.check_attn(out, ref, "static workspace, first call")
    # second call right after it: another shape (fewer partials than the array now holds) and other inputs
    b = build_case(882, 2, 2, 2, 700, c=4)
    lens_b = [700, 333]
    out2, ref2 = run_both(b, lens_b)
    H.check_attn(out2, ref2, "static workspace, second call")
    # and both agree with the oracle, not only with each other
    for case, lens, got in ((a, lens_a, out), (b, lens_b, out2)):
        q, kc_rm, vc_rm, kcb, vcb = case["host"]
        want = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32),
                                   128 ** -0.5, case["c"], case["b"])
        H.check_attn(got, want, "static workspace vs oracle")


def test_static_workspace_rejects_shapes_beyond_its_size():
    # Partials of this shape need more than the built-in array: a clear error and nothing launched.  The
    # call goes through the raw C symbol, because the Python wrapper would (rightly) refuse the undersized
    # code buffers first: they are never read, the size check comes before any launch.
    import ctypes
    n_seq, n_q, n_kv, cap = 64, 32, 8, 600000
    need = cq.cq_decode_attn_workspace_bytes(n_seq, n_q, n_kv, 128, 8, 8, cap)
    from paper_2405_03917_b200.binding import STATIC_WORKSPACE_BYTES
    assert need > STATIC_WORKSPACE_BYTES
    q = torch.zeros(n_seq, n_q, 128, dtype=torch.float16, device=DEV)
    cb = torch.zeros(n_kv, 16, 256, 8, dtype=torch.float32, device=DEV)
    codes = torch.zeros(16, dtype=torch.uint8, device=DEV)          # never read: the call must fail first
    sl = torch.zeros(n_seq, dtype=torch.int32, device=DEV)
    out = torch.zeros(n_seq, n_q, 128, dtype=torch.float32, device=DEV)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    st = cq.lib().cq_decode_attn_static(p(q), p(codes), p(codes), p(cb), p(cb), p(sl), 1.0, n_seq, n_q, n_kv, 128, 8, 8,
                                        cap, p(out), None)
    assert st == -5                      # CQ_ERR_WORKSPACE
    torch.cuda.synchronize()
    with pytest.raises(ValueError):      # and the wrapper checks the buffers against the shape
        cq.cq_decode_attn_static(q, codes, codes, cb, cb, sl, 1.0, 8, 8, cap, out)
