"""GPU parity of cq_prefill_attn (causal attention of a run of new tokens over the coded cache)
against the fp64 CPU oracle: both kernels, MHA and GQA, every group size of the tensor-core
kernel, ragged and short contexts, queries without a position, and the agreement of its last
row with the single-query decode attention."""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def to_lib(rm, D, c, b):
    t = torch.from_numpy(rm.astype(np.uint8)) if b <= 8 else torch.from_numpy(rm.astype(np.uint16).view(np.int16))
    return cq.cq_codes_from_rowmajor(t.to(DEV), D, c, b)


def random_case(seed, c, b, n_q, Hq, Hkv, lens, cap, D=128):
    rng = np.random.default_rng(seed)
    G = D // c
    kcb, vcb = (torch.from_numpy(rng.standard_normal((Hkv, G, 1 << b, c)).astype(np.float32)) for _ in range(2))
    q = torch.from_numpy(rng.standard_normal((len(lens), n_q, Hq, D)).astype(np.float16))
    kc_rm = rng.integers(0, 1 << b, size=(len(lens), cap, Hkv, G)).astype(np.int32)
    vc_rm = rng.integers(0, 1 << b, size=(len(lens), cap, Hkv, G)).astype(np.int32)
    return q, kc_rm, vc_rm, kcb, vcb


def run_both(q, kc_rm, vc_rm, kcb, vcb, lens, scale, c, b, variant):
    n_seq, cap, Hkv, G = kc_rm.shape
    D = G * c
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = cq.cq_prefill_attn(q.to(DEV), to_lib(kc_rm, D, c, b), to_lib(vc_rm, D, c, b), kcb.to(DEV), vcb.to(DEV), sl,
                             scale, c, b, cap, variant=variant)
    ref = oracle.prefill_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), scale, c, b)
    return out.cpu().numpy(), ref


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("c,n_q,Hq,Hkv,lens", [
    (8, 16, 4, 1, [700, 33, 16]),            # GQA R = 4: one row tile
    (8, 37, 2, 2, [300, 37, 64]),            # MHA, three row tiles, a prompt that is the whole cache
    (4, 20, 8, 2, [129, 1000]),              # R = 4, 32 groups
    (2, 9, 2, 1, [65, 9]),                   # R = 2, 64 groups
    (8, 5, 32, 1, [200, 5]),                 # R = 32: two queries per row tile
])
def test_prefill_matches_oracle(variant, c, n_q, Hq, Hkv, lens):
    cap = max(lens) + 3
    q, kc_rm, vc_rm, kcb, vcb = random_case(100 + c + n_q, c, 8, n_q, Hq, Hkv, lens, cap)
    got, ref = run_both(q, kc_rm, vc_rm, kcb, vcb, lens, 1 / np.sqrt(128), c, 8, variant)
    for s in range(len(lens)):
        H.check_attn(got[s], ref[s], f"c={c} seq {s} variant {variant}")


@pytest.mark.parametrize("variant", [1, 2])
def test_queries_without_a_position_give_zero_rows(variant):
    # 7 queries, but sequence 1 caches 4 tokens and sequence 2 none: their first queries attend nothing
    lens = [50, 4, 0]
    q, kc_rm, vc_rm, kcb, vcb = random_case(7, 8, 8, 7, 4, 2, lens, 50)
    got, ref = run_both(q, kc_rm, vc_rm, kcb, vcb, lens, 0.1, 8, 8, variant)
    assert (got[1, :3] == 0).all() and (got[2] == 0).all()
    H.check_attn(got, ref, "short caches")


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("scale", [-0.07, 0.0])
def test_scales_that_are_not_positive(variant, scale):
    # a negative scale turns the order of the scores around (the kernel's shortcut for tiles below the causal limit
    # takes the maximum of the raw scores and must not be used), a zero scale gives the plain mean of the values
    lens = [400, 130]
    q, kc_rm, vc_rm, kcb, vcb = random_case(11, 8, 8, 12, 4, 1, lens, 400)
    got, ref = run_both(q, kc_rm, vc_rm, kcb, vcb, lens, scale, 8, 8, variant)
    H.check_attn(got, ref, f"scale {scale}")


def test_generic_kernel_covers_other_shapes():
    # head_dim 64 with 5-bit codes, and codes wider than a byte: no tensor-core kernel, the plain one serves
    for (D, c, b, Hq, Hkv) in [(64, 4, 5, 4, 2), (128, 8, 10, 2, 1), (32, 1, 3, 3, 3)]:
        lens = [40, 11]
        q, kc_rm, vc_rm, kcb, vcb = random_case(D + b, c, b, 6, Hq, Hkv, lens, 41, D=D)
        got, ref = run_both(q, kc_rm, vc_rm, kcb, vcb, lens, 0.2, c, b, 0)
        H.check_attn(got, ref, f"D={D} c={c} b={b}")
        with pytest.raises(cq.CQError):
            run_both(q, kc_rm, vc_rm, kcb, vcb, lens, 0.2, c, b, 2)


@pytest.mark.parametrize("variant", [1, 2])
def test_last_row_equals_decode_attention(variant):
    # the newest token's row is Eq. 1 for one query over the whole cache: what cq_decode_attn computes
    w = H.small_workload("prefill_vs_decode", 0, 8, 8, 3, 8, 2, 1500)
    lens = [1500, 777, 64]
    n_q = 24
    xk = synth.layer_activations(w, 0, False, 3, 1500)
    xv = synth.layer_activations(w, 0, True, 3, 1500)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, 8, 8)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, 8, 8)
    g = torch.Generator().manual_seed(5)
    q = torch.randn(3, n_q, 8, 128, generator=g).to(torch.float16)
    got, ref = run_both(q, kc_rm, vc_rm, kcb, vcb, lens, (1 / np.sqrt(128)), 8, 8, variant)
    for s in range(3):
        H.check_attn(got[s], ref[s], f"seq {s}")
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    dec = cq.cq_decode_attn(q[:, -1].contiguous().to(DEV), to_lib(kc_rm, 128, 8, 8), to_lib(vc_rm, 128, 8, 8),
                            kcb.to(DEV), vcb.to(DEV), sl, (1 / np.sqrt(128)), 8, 8, 1500).cpu().numpy()
    H.check_attn(got[:, -1], dec, "last row vs decode")


def test_bad_arguments_are_refused():
    q, kc_rm, vc_rm, kcb, vcb = random_case(3, 8, 8, 4, 2, 2, [10], 10)
    sl = torch.tensor([10], dtype=torch.int32, device=DEV)
    kb, vb = to_lib(kc_rm, 128, 8, 8), to_lib(vc_rm, 128, 8, 8)
    with pytest.raises(cq.CQError):                      # more queries than the cache can hold
        cq.cq_prefill_attn(torch.zeros(1, 11, 2, 128, dtype=torch.float16, device=DEV), kb, vb, kcb.to(DEV), vcb.to(DEV),
                           sl, 0.1, 8, 8, 10)
    with pytest.raises(ValueError):                      # undersized code buffer
        cq.cq_prefill_attn(q.to(DEV), kb[:16], vb, kcb.to(DEV), vcb.to(DEV), sl, 0.1, 8, 8, 10)
