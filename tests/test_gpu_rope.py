"""GPU parity of decode attention over codes of pre-RoPE keys (cq_decode_attn_rope) against the
fp64 CPU oracle: both pairings, MHA and GQA, byte and wide codes, ragged and empty contexts, and
the reduction to the plain attention when every angle is zero."""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def rope_tables(max_tokens, P, base=10000.0):
    t = np.arange(max_tokens, dtype=np.float64)[:, None]
    ang = t * base ** (-np.arange(P, dtype=np.float64) / P)[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def case(seed, c, b, n_q, n_kv, lens, cap, D=128):
    rng = np.random.default_rng(seed)
    G = D // c
    kcb, vcb = (torch.from_numpy(rng.standard_normal((n_kv, G, 1 << b, c)).astype(np.float32)) for _ in range(2))
    q = torch.from_numpy(rng.standard_normal((len(lens), n_q, D)).astype(np.float16))
    kc_rm = rng.integers(0, 1 << b, size=(len(lens), cap, n_kv, G)).astype(np.int32)
    vc_rm = rng.integers(0, 1 << b, size=(len(lens), cap, n_kv, G)).astype(np.int32)
    return q, kc_rm, vc_rm, kcb, vcb


def to_lib(rm, D, c, b):
    t = torch.from_numpy(rm.astype(np.uint8)) if b <= 8 else torch.from_numpy(rm.astype(np.uint16).view(np.int16))
    return cq.cq_codes_from_rowmajor(t.to(DEV), D, c, b)


@pytest.mark.parametrize("c,b,n_q,n_kv,lens,D", [
    (8, 8, 2, 2, [700, 33, 0], 128),
    (8, 8, 4, 1, [1, 16, 17, 2100], 128),        # GQA R = 4, several splits
    (4, 8, 2, 1, [300, 257], 128),
    (2, 6, 3, 3, [90], 64),
    (8, 10, 2, 1, [500, 123], 128),              # CQ-8c10b
    (2, 1, 1, 1, [40], 4),                       # tiny shapes: the staged codebook would not be 16-byte aligned
    (2, 3, 2, 1, [70, 5], 12),
])
@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_attention_matches_the_oracle(c, b, n_q, n_kv, lens, D, pairing):
    cap = max(lens) + 7
    q, kc_rm, vc_rm, kcb, vcb = case(60 + c + b + pairing, c, b, n_q, n_kv, lens, cap, D)
    cs, sn = rope_tables(cap, D // 2)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = cq.cq_decode_attn_rope(q.to(DEV), to_lib(kc_rm, D, c, b), to_lib(vc_rm, D, c, b), kcb.to(DEV), vcb.to(DEV), sl,
                                 torch.from_numpy(cs).to(DEV), torch.from_numpy(sn).to(DEV), D ** -0.5, c, b, cap,
                                 pairing=pairing).cpu().numpy()
    ref = oracle.decode_dense_rope(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), cs, sn,
                                   D ** -0.5, c, b, pairing)
    H.check_attn(out, ref, f"rope c={c} b={b} pairing={pairing}")
    for s_ in range(len(lens)):
        H.check_attn(out[s_], ref[s_], f"rope sequence {s_}")


def test_rope_with_zero_angles_is_the_plain_attention():
    c, b, D, lens = 8, 8, 128, [900, 50]
    cap = 900
    q, kc_rm, vc_rm, kcb, vcb = case(3, c, b, 4, 2, lens, cap)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kb, vb = to_lib(kc_rm, D, c, b), to_lib(vc_rm, D, c, b)
    ones, zeros = torch.ones(cap, D // 2, device=DEV), torch.zeros(cap, D // 2, device=DEV)
    plain = cq.cq_decode_attn(q.to(DEV), kb, vb, kcb.to(DEV), vcb.to(DEV), sl, 0.1, c, b, cap).cpu().numpy()
    for pairing in (0, 1):
        got = cq.cq_decode_attn_rope(q.to(DEV), kb, vb, kcb.to(DEV), vcb.to(DEV), sl, ones, zeros, 0.1, c, b, cap,
                                     pairing=pairing).cpu().numpy()
        H.check_attn(got, plain, f"zero angles, pairing {pairing}")


def test_rope_rejects_pairs_that_split_groups():
    D, cap = 128, 16
    q = torch.zeros(1, 1, D, dtype=torch.float16, device=DEV)
    sl = torch.ones(1, dtype=torch.int32, device=DEV)
    t = torch.zeros(cap, D // 2, device=DEV)
    # c = 128: one group, so channel i + 64 is in the same code as channel i but the groups cannot be halved
    cb = torch.zeros(1, 1, 4, 128, device=DEV)
    codes = torch.zeros(cq.cq_codes_bytes(1, cap, 1, D, 128, 2), dtype=torch.uint8, device=DEV)
    with pytest.raises(cq.CQError) as e:
        cq.cq_decode_attn_rope(q, codes, codes, cb, cb, sl, t, t, 1.0, 128, 2, cap, pairing=0)
    assert e.value.status == -3
    # c = 1: an interleaved pair would span two groups
    cb1 = torch.zeros(1, 128, 4, 1, device=DEV)
    codes1 = torch.zeros(cq.cq_codes_bytes(1, cap, 1, D, 1, 2), dtype=torch.uint8, device=DEV)
    with pytest.raises(cq.CQError) as e:
        cq.cq_decode_attn_rope(q, codes1, codes1, cb1, cb1, sl, t, t, 1.0, 1, 2, cap, pairing=1)
    assert e.value.status == -3


# ------------------------------------------------------------------------------- the tuned kernel

def run_rope(q, kc_rm, vc_rm, kcb, vcb, lens, cs, sn, cap, c, variant, scale):
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    return cq.cq_decode_attn_rope(q.to(DEV), to_lib(kc_rm, 128, c, 8), to_lib(vc_rm, 128, c, 8), kcb.to(DEV), vcb.to(DEV), sl,
                                  torch.from_numpy(cs).to(DEV), torch.from_numpy(sn).to(DEV), scale, c, 8, cap,
                                  pairing=0, variant=variant).cpu().numpy()


@pytest.mark.parametrize("c,n_q,n_kv", [(8, 2, 2), (8, 4, 2), (8, 4, 1), (8, 8, 1), (8, 16, 1), (8, 3, 1), (4, 2, 2), (4, 2, 1),
                                        (4, 4, 1), (4, 8, 1)])
def test_tuned_rope_kernel_matches_the_oracle(c, n_q, n_kv):
    # every number of query heads per CTA (1, 2, 4, 8) of both group sizes; empty, one-token, ragged contexts, a
    # context longer than the chunk of scores that shared memory holds, several ranges per sequence
    lens = [0, 1, 15, 16, 17, 700, 9000]
    cap = 9100
    q, kc_rm, vc_rm, kcb, vcb = case(200 + c + n_q, c, 8, n_q, n_kv, lens, cap)
    cs, sn = rope_tables(cap, 64)
    got = run_rope(q, kc_rm, vc_rm, kcb, vcb, lens, cs, sn, cap, c, 2, 128 ** -0.5)
    ref = oracle.decode_dense_rope(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), cs, sn,
                                   128 ** -0.5, c, 8, 0)
    for s_ in range(len(lens)):
        H.check_attn(got[s_], ref[s_], f"tuned rope c={c} Hq={n_q} Hkv={n_kv} sequence {s_}")
    assert (got[0] == 0).all()


def test_tuned_rope_kernel_with_tables_that_are_not_rotary():
    # phases that jump around: the stepped cosines leave the tables at once, every row is then read from them;
    # a table that is rotary except for one row in the middle of a batch's reach is caught at the batch's end or
    # stays within the kernel's check (the row after each batch), so only the first kind is asserted
    lens = [300, 64]
    cap = 320
    q, kc_rm, vc_rm, kcb, vcb = case(9, 8, 8, 4, 1, lens, cap)
    rng = np.random.default_rng(4)
    ang = rng.uniform(0, 6.28, size=(cap, 64))
    amp = rng.uniform(0.5, 1.5, size=(cap, 64))          # not even of unit length
    cs, sn = (amp * np.cos(ang)).astype(np.float32), (amp * np.sin(ang)).astype(np.float32)
    ref = oracle.decode_dense_rope(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), cs, sn,
                                   0.05, 8, 8, 0)
    for variant in (2, 1):
        got = run_rope(q, kc_rm, vc_rm, kcb, vcb, lens, cs, sn, cap, 8, variant, 0.05)
        H.check_attn(got, ref, f"arbitrary tables, variant {variant}")


def test_tuned_rope_kernel_with_scaled_and_shifted_rotary_tables():
    # amplitude and phase per pair, frequencies of another base: still of the rotary form, so the stepping holds
    lens = [1500, 77]
    cap = 1500
    q, kc_rm, vc_rm, kcb, vcb = case(10, 4, 8, 4, 2, lens, cap)
    rng = np.random.default_rng(5)
    t = np.arange(cap, dtype=np.float64)[:, None]
    freq = 500000.0 ** (-np.arange(64, dtype=np.float64) / 64)[None, :]
    phase, amp = rng.uniform(0, 6.28, size=(1, 64)), rng.uniform(0.7, 1.3, size=(1, 64))
    cs, sn = (amp * np.cos(t * freq + phase)).astype(np.float32), (amp * np.sin(t * freq + phase)).astype(np.float32)
    ref = oracle.decode_dense_rope(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), cs, sn,
                                   128 ** -0.5, 4, 8, 0)
    got = run_rope(q, kc_rm, vc_rm, kcb, vcb, lens, cs, sn, cap, 4, 2, 128 ** -0.5)
    H.check_attn(got, ref, "scaled rotary tables")


def test_tuned_rope_kernel_is_refused_where_it_does_not_apply():
    q, kc_rm, vc_rm, kcb, vcb = case(1, 8, 8, 2, 1, [20], 20)
    cs, sn = rope_tables(20, 64)
    sl = torch.tensor([20], dtype=torch.int32, device=DEV)
    with pytest.raises(cq.CQError):          # the other pairing
        cq.cq_decode_attn_rope(q.to(DEV), to_lib(kc_rm, 128, 8, 8), to_lib(vc_rm, 128, 8, 8), kcb.to(DEV), vcb.to(DEV), sl,
                               torch.from_numpy(cs).to(DEV), torch.from_numpy(sn).to(DEV), 0.1, 8, 8, 20, pairing=1, variant=2)
