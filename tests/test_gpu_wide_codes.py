"""GPU parity for codes wider than a byte (b = 9, 10, 12; CQ-8c10b of Section 4 is b = 10):
encode, the documented layout of the packed upper bits, appends into blocks that other tokens
share, decode attention, and centroid learning, each against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def to_dev_rowmajor(rm_np):
    """int codes (n_seq, cap, n_heads, G) -> int16 CUDA tensor holding the unsigned 16-bit patterns."""
    return torch.from_numpy(np.ascontiguousarray(rm_np).astype(np.uint16).view(np.int16)).to(DEV)


def from_dev_rowmajor(t):
    return t.cpu().numpy().view(np.uint16).astype(np.int32)


def encode_rowmajor(x, cb, c, b, cap, **kw):
    n_seq, n_tokens, n_heads, D = x.shape
    buf = torch.zeros(cq.cq_codes_bytes(n_seq, cap, n_heads, D, c, b), dtype=torch.uint8, device=DEV)
    cq.cq_encode(x.to(DEV), cb.to(DEV), c, b, buf, cap, **kw)
    return buf, from_dev_rowmajor(cq.cq_codes_to_rowmajor(buf, n_seq, cap, n_heads, D, c, b))


@pytest.mark.parametrize("c,b,head_dim,n_heads,n_tokens", [(8, 10, 128, 2, 70), (8, 9, 128, 1, 33), (4, 12, 32, 2, 21),
                                                         (8, 10, 64, 3, 16), (16, 10, 128, 1, 50), (4, 10, 128, 2, 300),
                                                         (2, 9, 128, 1, 130), (8, 12, 128, 1, 90)])
def test_encode_wide_codes(c, b, head_dim, n_heads, n_tokens):
    xk, xv, kcb, vcb, _ = H.generic_case(900 + b + c, 2, n_tokens, n_heads, n_heads, head_dim, c, b)
    tuned = head_dim == 128 and c in (2, 4, 8) and b in (9, 10, 12)      # chunks of 256 centroids on the tensor cores
    small = (1 << b) * c * 4 + 8 * c * 4 <= 48 * 1024
    for x, cb in ((xk, kcb), (xv, vcb)):
        for variant in (1, 0) + ((2,) if tuned else ()) + ((3,) if small else ()):
            _, rm = encode_rowmajor(x, cb, c, b, n_tokens, variant=variant)
            assert rm.max() >= 256                                    # the upper bits are in use
            H.check_codes(x.numpy().reshape(-1, n_heads, head_dim), cb.numpy(), rm.reshape(-1, n_heads, head_dim // c), c, b)


def test_encode_8c10b_bulk_and_duplicate_centroids_across_chunks():
    # enough vectors for the 64-per-warp form of the tuned kernel; centroids duplicated in a later chunk of 256
    # must lose the tie to their first copy (lowest index)
    c, b, D, nh, n_tok = 8, 10, 128, 8, 2500
    g = torch.Generator().manual_seed(12)
    cb = torch.randn(nh, D // c, 1 << b, c, generator=g)
    cb[:, :, 700] = cb[:, :, 40]
    cb[:, :, 300] = cb[:, :, 299]
    x = torch.randn(8, n_tok, nh, D, generator=g).to(torch.float16)
    x[0, :64, :, :] = cb[:, :, 40].reshape(1, nh, D).to(torch.float16)          # vectors that sit (nearly) on centroid 40 / 700
    for variant in (2, 1):
        _, rm = encode_rowmajor(x, cb, c, b, n_tok, variant=variant)
        assert not (rm == 700).any() and not (rm == 300).any()
        H.check_codes(x.numpy().reshape(-1, nh, D), cb.numpy(), rm.reshape(-1, nh, D // c), c, b)


@pytest.mark.parametrize("b", [9, 10, 12, 16])
def test_layout_of_the_packed_upper_bits(b):
    n_seq, cap, nh, D, c = 2, 37, 3, 64, 8
    G, hb = D // c, b - 8
    rng = np.random.default_rng(b)
    rm = rng.integers(0, 1 << b, size=(n_seq, cap, nh, G)).astype(np.int32)
    buf = cq.cq_codes_from_rowmajor(to_dev_rowmajor(rm), D, c, b)
    NB = (cap + 15) // 16
    assert buf.numel() == cq.cq_codes_bytes(n_seq, cap, nh, D, c, b) == -(-n_seq * nh * NB * G * (16 + 2 * hb) // 16) * 16
    back = from_dev_rowmajor(cq.cq_codes_to_rowmajor(buf, n_seq, cap, nh, D, c, b))
    assert np.array_equal(back, rm)
    host = buf.cpu().numpy()
    for (s, t, h, g) in [(0, 0, 0, 0), (1, 36, 2, G - 1), (0, 17, 1, 3), (1, 16, 0, 5), (0, 15, 2, 7)]:
        block = ((s * nh + h) * NB + t // 16) * G * (16 + 2 * hb)
        assert host[block + g * 16 + t % 16] == rm[s, t, h, g] & 255
        word = int.from_bytes(host[block + G * 16 + g * 2 * hb: block + G * 16 + (g + 1) * 2 * hb].tobytes(), "little")
        assert (word >> ((t % 16) * hb)) & ((1 << hb) - 1) == rm[s, t, h, g] >> 8


def test_append_into_shared_upper_words():
    # appended tokens land in blocks whose upper-bit words already hold other tokens' bits
    c, b, D, nh, cap = 8, 10, 128, 2, 70
    xk, _, kcb, _, _ = H.generic_case(31, 3, cap, nh, nh, D, c, b)
    full, rm_full = encode_rowmajor(xk, kcb, c, b, cap)
    buf = torch.zeros_like(full)
    cq.cq_encode(xk[:, :40].contiguous().to(DEV), kcb.to(DEV), c, b, buf, cap)
    cq.cq_encode(xk[:, 40:].contiguous().to(DEV), kcb.to(DEV), c, b, buf, cap, token_offset=40)
    assert torch.equal(buf, full)
    # overwrite single positions (old bits must go, neighbours must stay)
    buf2 = full.clone()
    offs = torch.tensor([5, 69, 0], dtype=torch.int32, device=DEV)
    cq.cq_encode(xk[:, 10:11].contiguous().to(DEV), kcb.to(DEV), c, b, buf2, cap, seq_offsets=offs)
    rm2 = from_dev_rowmajor(cq.cq_codes_to_rowmajor(buf2, 3, cap, nh, D, c, b))
    want = rm_full.copy()
    for s, p in enumerate([5, 69, 0]):
        want[s, p] = rm_full[s, 10]
    assert np.array_equal(rm2, want)


def random_attention_case(seed, c, b, n_q, n_kv, lens, cap, D=128):
    rng = np.random.default_rng(seed)
    G, n_seq = D // c, len(lens)
    kcb, vcb = (torch.from_numpy(rng.standard_normal((n_kv, G, 1 << b, c)).astype(np.float32)) for _ in range(2))
    q = torch.from_numpy(rng.standard_normal((n_seq, n_q, D)).astype(np.float16))
    kc_rm = rng.integers(0, 1 << b, size=(n_seq, cap, n_kv, G)).astype(np.int32)
    vc_rm = rng.integers(0, 1 << b, size=(n_seq, cap, n_kv, G)).astype(np.int32)
    return q, kc_rm, vc_rm, kcb, vcb


def attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, scale, c, b, variant):
    n_seq, cap, n_kv, G = kc_rm.shape
    D = G * c
    kb = cq.cq_codes_from_rowmajor(to_dev_rowmajor(kc_rm), D, c, b)
    vb = cq.cq_codes_from_rowmajor(to_dev_rowmajor(vc_rm), D, c, b)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = cq.cq_decode_attn(q.to(DEV), kb, vb, kcb.to(DEV), vcb.to(DEV), sl, scale, c, b, cap, variant=variant)
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), scale, c, b)
    return out.cpu().numpy(), ref


@pytest.mark.parametrize("c,b,n_q,n_kv,lens", [
    (8, 10, 2, 2, [700, 33, 0]),               # CQ-8c10b, MHA
    (8, 10, 4, 1, [1, 16, 17, 1200]),          # GQA R = 4
    (8, 10, 3, 3, [15, 2049, 128, 2048]),      # block and round edges of the tuned kernel
    (8, 9, 2, 1, [300, 257]),
    (16, 10, 1, 1, [500]),
])
def test_attention_wide_codes(c, b, n_q, n_kv, lens):
    D, cap = 128, max(lens) + 5
    q, kc_rm, vc_rm, kcb, vcb = random_attention_case(40 + b + n_q, c, b, n_q, n_kv, lens, cap)
    for variant in (1, 0):                      # generic; automatic (the tuned kernel for 8c10b)
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, D ** -0.5, c, b, variant)
        H.check_attn(out, ref, f"c={c} b={b} Hq={n_q} Hkv={n_kv} variant={variant}")
        for s_ in range(len(lens)):
            H.check_attn(out[s_], ref[s_], f"sequence {s_} variant={variant}")


def test_attention_8c10b_long_contexts_and_several_chunks():
    # few items, so the launch plan cuts the contexts into chunks of a few rounds; ragged ends
    lens = [9000, 4097, 20000]
    q, kc_rm, vc_rm, kcb, vcb = random_attention_case(5, 8, 10, 2, 1, lens, 20011)
    out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, 128 ** -0.5, 8, 10, 2)
    H.check_attn(out, ref, "8c10b long")
    for s_ in range(3):
        H.check_attn(out[s_], ref[s_], f"8c10b long, sequence {s_}")


def test_attention_8c10b_weight_unit_is_coarsened():
    # zero query (every weight is the maximum), scores rising along the context, scores falling
    c, b, cap, n_kv, n_q = 8, 10, 20000, 1, 2
    q, kc_rm, vc_rm, kcb, vcb = random_attention_case(6, c, b, n_q, n_kv, [cap] * 3, cap)
    q[0] = 0
    q[2] = q[1]
    kc_rm[1] = kc_rm[2]
    vc_rm[1] = vc_rm[2]
    khat = oracle.dequant(kc_rm[1].reshape(cap, n_kv, -1), kcb.numpy(), c, b)[:, 0]
    order = np.argsort(khat @ q[1, 0].double().numpy(), kind="stable")
    kc_rm[2], vc_rm[2] = kc_rm[1][order[::-1]], vc_rm[1][order[::-1]]
    kc_rm[1], vc_rm[1] = kc_rm[1][order], vc_rm[1][order]
    for variant in (1, 2):
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [cap, cap - 3, cap - 17], 0.7, c, b, variant)
        H.check_attn(out, ref, f"flat/rising/falling variant={variant}")
        for s_ in range(3):
            H.check_attn(out[s_], ref[s_], f"flat/rising/falling sequence {s_} variant={variant}")


def test_attention_8c10b_spread_tail():
    # 152 (sequence, query head) items on 148 SMs: the last four are spread over several CTAs each
    lens = [int(v) for v in np.random.default_rng(8).integers(1, 8200, size=18)] + [8200]
    q, kc_rm, vc_rm, kcb, vcb = random_attention_case(9, 8, 10, 8, 2, lens, 8200)
    out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, 128 ** -0.5, 8, 10, 2)
    H.check_attn(out, ref, "8c10b spread tail")
    H.check_attn(out[-1], ref[-1], "8c10b spread tail, last sequence")


def test_encode_then_attention_8c10b_end_to_end():
    # the codes the attention reads are the oracle's; the CUDA codes are checked against them first
    c, b, D, n_q, n_kv, n_tok = 8, 10, 128, 2, 1, 600
    xk, xv, kcb, vcb, q = H.generic_case(77, 2, n_tok, n_q, n_kv, D, c, b)
    kc_rm, kres = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, vres = H.oracle_encode_rowmajor(xv, vcb, c, b)
    for x, cb, res in ((xk, kcb, kres), (xv, vcb, vres)):
        _, rm = encode_rowmajor(x, cb, c, b, n_tok)
        H.check_codes(x.numpy().reshape(-1, n_kv, D), cb.numpy(), rm.reshape(-1, n_kv, D // c), c, b, res)
    kb = cq.cq_codes_from_rowmajor(to_dev_rowmajor(kc_rm), D, c, b)
    vb = cq.cq_codes_from_rowmajor(to_dev_rowmajor(vc_rm), D, c, b)
    lens = [n_tok, n_tok - 77]
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = cq.cq_decode_attn(q.to(DEV), kb, vb, kcb.to(DEV), vcb.to(DEV), sl, D ** -0.5, c, b, n_tok).cpu().numpy()
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), D ** -0.5, c, b)
    H.check_attn(out, ref, "8c10b end to end")


def test_centroid_learning_with_1024_centroids():
    c, b, n_heads, n_vec = 8, 10, 1, 2500
    g = torch.Generator().manual_seed(9)
    x = (torch.randn(n_vec, n_heads, 128, generator=g) * 1.5).to(torch.float16)
    G = 128 // c
    u = np.random.default_rng(10).random((n_heads, G, 1 << b))
    want0, _ = oracle.kmeanspp_init(x.numpy(), None, u, c, b)
    got0 = cq.cq_kmeanspp_init(x.to(DEV), None, torch.from_numpy(u).to(DEV), c, b).cpu().numpy()
    assert np.array_equal(got0, want0)
    want, _, obj = oracle.lloyd_step(x.numpy(), None, want0, c, b)
    got, gobj = cq.cq_lloyd_step(x.to(DEV), None, torch.from_numpy(want0).to(DEV), c, b)
    got, gobj = got.cpu().numpy(), gobj.cpu().numpy()
    close = np.abs(got - want) <= 2e-5 * np.abs(want).max() + 2e-5 * np.abs(want)
    assert close.mean() > 0.999
    np.testing.assert_allclose(gobj, obj, rtol=1e-5)
