"""GPU parity tests: the CUDA library (through its C ABI) against the fp64 CPU oracle,
element by element, on the same seeded inputs.  Sizes here are ones the oracle finishes
in seconds; the full-size workloads are in test_gpu_full_size.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def encode_both(x, cb, c, b, max_tokens, variant=0, token_offset=0):
    """x (n_seq, n_tokens, n_heads, D) fp16 CPU, cb fp32 CPU -> (gpu rowmajor codes np, oracle triple)."""
    n_seq, n_tokens, n_heads, D = x.shape
    buf = torch.zeros(cq.cq_codes_bytes(n_seq, max_tokens, n_heads, D, c, b), dtype=torch.uint8, device=DEV)
    cq.cq_encode(x.to(DEV), cb.to(DEV), c, b, buf, max_tokens, token_offset=token_offset, variant=variant)
    rm = cq.cq_codes_to_rowmajor(buf, n_seq, max_tokens, n_heads, D, c, b).cpu().numpy()
    return buf, rm


# ------------------------------------------------------------------------------- encode

@pytest.mark.parametrize("variant", [1, 0])
def test_config0_encode_bit_exact(variant):
    w = synth.WORKLOADS[0]
    ties = 0
    for is_v in (False, True):
        x = synth.layer_activations(w, 0, is_v, w.n_seq, w.n_tokens)
        cb = synth.layer_codebooks(w, 0, is_v)
        _, rm = encode_both(x, cb, w.c, w.b, w.n_tokens, variant)
        n, total = H.check_codes(x.numpy().reshape(-1, 1, 128), cb.numpy(), rm.reshape(-1, 1, w.G), w.c, w.b)
        ties += n
    assert ties <= 2 * 1024 * 16 // 1000          # near-ties are rare


@pytest.mark.parametrize("c,b,head_dim,n_heads,n_tokens", [
    (2, 8, 128, 3, 100), (4, 8, 128, 2, 77), (8, 8, 128, 2, 130), (1, 4, 64, 2, 33), (16, 8, 128, 1, 50),
    (8, 5, 64, 3, 47), (4, 1, 32, 2, 19), (8, 8, 256, 1, 40), (2, 3, 16, 5, 16),
])
def test_encode_shapes_and_ragged_tails(c, b, head_dim, n_heads, n_tokens):
    xk, xv, kcb, vcb, _ = H.generic_case(11 * c + b, 2, n_tokens, n_heads, n_heads, head_dim, c, b)
    tuned = head_dim == 128 and b == 8 and c in (2, 4, 8)
    for x, cb in ((xk, kcb), (xv, vcb)):
        for variant in (1, 0, 3) + ((2, 4) if tuned else ()):     # generic, automatic, few-vector, tuned, tensor-memory
            _, rm = encode_both(x, cb, c, b, n_tokens, variant)
            H.check_codes(x.numpy().reshape(-1, n_heads, head_dim), cb.numpy(),
                          rm.reshape(-1, n_heads, head_dim // c), c, b)


def test_encode_codebook_contains_inputs_and_exact_ties():
    # inputs equal to centroids -> that centroid's lowest index; duplicated centroids -> lowest index
    c, b, D, H_ = 8, 8, 128, 2
    g = torch.Generator().manual_seed(5)
    cb = torch.randn(H_, D // c, 256, c, generator=g).to(torch.float16).to(torch.float32)
    cb[:, :, 200] = cb[:, :, 7]
    pick = torch.randint(0, 256, (1, 64, H_, D // c), generator=g)
    hh = torch.arange(H_)[None, :, None]
    gg = torch.arange(D // c)[None, None, :]
    x = cb[hh, gg, pick[0]].reshape(1, 64, H_, D)        # group g of token t = centroid pick[t, h, g]
    for variant in (1, 0, 2, 3, 4):
        _, rm = encode_both(x.to(torch.float16), cb, c, b, 64, variant)
        want = torch.where(pick == 200, torch.tensor(7), pick).numpy()
        assert np.array_equal(rm.astype(np.int64), want)


@pytest.mark.parametrize("c,n_seq,n_tokens,n_heads", [(8, 2, 700, 3), (2, 1, 1300, 2), (4, 3, 257, 2), (8, 1, 9, 1)])
def test_tensor_memory_encode_kernel(c, n_seq, n_tokens, n_heads):
    # several 256-vector tiles with a ragged last one, groups split over CTAs, sequences that end inside a tile
    xk, xv, kcb, vcb, _ = H.generic_case(900 + c + n_tokens, n_seq, n_tokens, n_heads, n_heads, 128, c, 8)
    for x, cb in ((xk, kcb), (xv, vcb)):
        _, rm = encode_both(x, cb, c, 8, n_tokens, 4)
        H.check_codes(x.numpy().reshape(-1, n_heads, 128), cb.numpy(), rm.reshape(-1, n_heads, 128 // c), c, 8)
    # the key and the value in one launch, appended behind per-sequence offsets
    cap = n_tokens + 40
    nbytes = cq.cq_codes_bytes(n_seq, cap, n_heads, 128, c, 8)
    want_k, want_v, got_k, got_v = (torch.zeros(nbytes, dtype=torch.uint8, device=DEV) for _ in range(4))
    offs = torch.arange(n_seq, dtype=torch.int32, device=DEV) * 13
    cq.cq_encode(xk.to(DEV), kcb.to(DEV), c, 8, want_k, cap, seq_offsets=offs, variant=1)
    cq.cq_encode(xv.to(DEV), vcb.to(DEV), c, 8, want_v, cap, seq_offsets=offs, variant=1)
    cq.cq_encode(xk.to(DEV), kcb.to(DEV), c, 8, got_k, cap, seq_offsets=offs, variant=4)
    cq.cq_encode(xv.to(DEV), vcb.to(DEV), c, 8, got_v, cap, seq_offsets=offs, variant=4)
    assert torch.equal(got_k, want_k) and torch.equal(got_v, want_v)


def test_tensor_memory_encode_codebooks_fp16_cannot_carry():
    # centroids beyond the fp16 range in one group, huge norms in another: those groups are encoded the exact way
    c, n_heads, n_tokens = 8, 2, 300
    xk, _, kcb, _, _ = H.generic_case(77, 1, n_tokens, n_heads, n_heads, 128, c, 8)
    kcb = kcb.clone()
    kcb[0, 3] *= 30000.0
    kcb[1, 5, 17] = 250.0
    kcb[1, 9] *= 1e-6
    for variant in (4, 2):
        _, rm = encode_both(xk, kcb, c, 8, n_tokens, variant)
        H.check_codes(xk.numpy().reshape(-1, n_heads, 128), kcb.numpy(), rm.reshape(-1, n_heads, 128 // c), c, 8)


def test_bulk_encode_takes_the_same_codes_on_every_path():
    # enough vectors that the automatic choice is the bulk kernel (key and value in one launch as well)
    c, n_heads, n_tokens = 8, 32, 4800
    g = torch.Generator().manual_seed(31)
    xk = torch.randn(1, n_tokens, n_heads, 128, generator=g).to(torch.float16)
    xv = (torch.randn(1, n_tokens, n_heads, 128, generator=g) * 0.3).to(torch.float16)
    kcb = torch.randn(n_heads, 16, 256, c, generator=g)
    vcb = torch.randn(n_heads, 16, 256, c, generator=g) * 0.3
    nbytes = cq.cq_codes_bytes(1, n_tokens, n_heads, 128, c, 8)
    bufs = {}
    for variant in (0, 2, 4):
        bufs[variant], _ = encode_both(xk, kcb, c, 8, n_tokens, variant)
    assert torch.equal(bufs[0], bufs[2]) and torch.equal(bufs[0], bufs[4])
    got_k, got_v = (torch.zeros(nbytes, dtype=torch.uint8, device=DEV) for _ in range(2))
    cq.cq_encode_kv(xk.to(DEV), xv.to(DEV), kcb.to(DEV), vcb.to(DEV), c, 8, got_k, got_v, n_tokens)
    want_v, _ = encode_both(xv, vcb, c, 8, n_tokens, 2)
    assert torch.equal(got_k, bufs[2]) and torch.equal(got_v, want_v)
    # a sample of the tokens against the oracle
    idx = np.random.default_rng(3).integers(0, n_tokens, size=64)
    rm = cq.cq_codes_to_rowmajor(got_k, 1, n_tokens, n_heads, 128, c, 8).cpu().numpy()[0, idx]
    H.check_codes(xk[0, idx].numpy(), kcb.numpy(), rm, c, 8)


def test_append_positions_and_untouched_bytes():
    c, b, D, nh, cap = 8, 8, 128, 2, 70
    xk, _, kcb, _, _ = H.generic_case(3, 3, cap, nh, nh, D, c, b)
    full, rm_full = encode_both(xk, kcb, c, b, cap)
    # prefill 40 tokens, then append tokens 40..69 one call of 30 tokens at offset 40
    buf = torch.full((cq.cq_codes_bytes(3, cap, nh, D, c, b),), 0, dtype=torch.uint8, device=DEV)
    cq.cq_encode(xk[:, :40].contiguous().to(DEV), kcb.to(DEV), c, b, buf, cap)
    cq.cq_encode(xk[:, 40:].contiguous().to(DEV), kcb.to(DEV), c, b, buf, cap, token_offset=40)
    assert torch.equal(buf, full)
    # per-sequence offsets: single-token append at positions (5, 69, 0); everything else untouched
    buf2 = full.clone()
    offs = torch.tensor([5, 69, 0], dtype=torch.int32, device=DEV)
    newtok = xk[:, 10:11].contiguous()
    cq.cq_encode(newtok.to(DEV), kcb.to(DEV), c, b, buf2, cap, seq_offsets=offs)
    rm2 = cq.cq_codes_to_rowmajor(buf2, 3, cap, nh, D, c, b).cpu().numpy()
    want = rm_full.copy()
    for s, p in enumerate([5, 69, 0]):
        want[s, p] = rm_full[s, 10]
    assert np.array_equal(rm2, want)
    # offsets past the capacity are skipped, not written out of bounds
    offs_bad = torch.tensor([cap, cap + 5, 3], dtype=torch.int32, device=DEV)
    buf3 = full.clone()
    cq.cq_encode(newtok.to(DEV), kcb.to(DEV), c, b, buf3, cap, seq_offsets=offs_bad)
    rm3 = cq.cq_codes_to_rowmajor(buf3, 3, cap, nh, D, c, b).cpu().numpy()
    want3 = rm_full.copy()
    want3[2, 3] = rm_full[2, 10]
    assert np.array_equal(rm3, want3)


@pytest.mark.parametrize("c,b,head_dim", [(8, 8, 128), (2, 8, 128), (4, 5, 64), (8, 10, 128)])
def test_encode_kv_equals_two_encodes(c, b, head_dim):
    nh, cap = 2, 50
    xk, xv, kcb, vcb, _ = H.generic_case(70 + c + b, 3, cap, nh, nh, head_dim, c, b)
    nbytes = cq.cq_codes_bytes(3, cap, nh, head_dim, c, b)
    want_k, want_v, got_k, got_v = (torch.zeros(nbytes, dtype=torch.uint8, device=DEV) for _ in range(4))
    offs = torch.tensor([3, 49, 0], dtype=torch.int32, device=DEV)
    for x, cb, buf in ((xk, kcb, want_k), (xv, vcb, want_v)):
        cq.cq_encode(x[:, :30].contiguous().to(DEV), cb.to(DEV), c, b, buf, cap)                      # prefill
        cq.cq_encode(x[:, 30:31].contiguous().to(DEV), cb.to(DEV), c, b, buf, cap, seq_offsets=offs)  # append
    cq.cq_encode_kv(xk[:, :30].contiguous().to(DEV), xv[:, :30].contiguous().to(DEV), kcb.to(DEV), vcb.to(DEV), c, b,
                    got_k, got_v, cap)
    cq.cq_encode_kv(xk[:, 30:31].contiguous().to(DEV), xv[:, 30:31].contiguous().to(DEV), kcb.to(DEV), vcb.to(DEV), c, b,
                    got_k, got_v, cap, seq_offsets=offs)
    assert torch.equal(got_k, want_k) and torch.equal(got_v, want_v)


def test_layout_roundtrip_matches_documented_offsets():
    n_seq, cap, nh, D, c, b = 2, 37, 3, 64, 4, 8
    G = D // c
    rm = torch.randint(0, 256, (n_seq, cap, nh, G), dtype=torch.uint8)
    buf = cq.cq_codes_from_rowmajor(rm.to(DEV), D, c, b)
    assert buf.numel() == cq.cq_codes_bytes(n_seq, cap, nh, D, c, b)
    back = cq.cq_codes_to_rowmajor(buf, n_seq, cap, nh, D, c, b).cpu()
    assert torch.equal(back, rm)
    host = buf.cpu().numpy()
    NB = (cap + 15) // 16
    for (s, t, h, g) in [(0, 0, 0, 0), (1, 36, 2, 15), (0, 17, 1, 3), (1, 16, 0, 9)]:
        off = (((s * nh + h) * NB + t // 16) * G + g) * 16 + t % 16
        assert host[off] == rm[s, t, h, g]


# ------------------------------------------------------------------------------- attention

def attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, scale, c, b, variant):
    """Codes are the ORACLE's (row-major int32 numpy); both sides read the same codes."""
    n_seq, cap, n_kv, G = kc_rm.shape
    D = G * c
    kb = cq.cq_codes_from_rowmajor(torch.from_numpy(kc_rm.astype(np.uint8)).to(DEV), D, c, b)
    vb = cq.cq_codes_from_rowmajor(torch.from_numpy(vc_rm.astype(np.uint8)).to(DEV), D, c, b)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    out = cq.cq_decode_attn(q.to(DEV), kb, vb, kcb.to(DEV), vcb.to(DEV), sl, scale, c, b, cap, variant=variant)
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32),
                              scale, c, b)
    return out.cpu().numpy(), ref


@pytest.mark.parametrize("variant", [1, 0])
def test_config0_end_to_end(variant):
    # encode K and V on the GPU, check codes; then attention on the oracle's codes
    w = synth.WORKLOADS[0]
    xk = synth.layer_activations(w, 0, False, 1, w.n_tokens)
    xv = synth.layer_activations(w, 0, True, 1, w.n_tokens)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(0, 0, 1, 1)
    kc_rm, kres = H.oracle_encode_rowmajor(xk, kcb, w.c, w.b)
    vc_rm, vres = H.oracle_encode_rowmajor(xv, vcb, w.c, w.b)
    _, gk = encode_both(xk, kcb, w.c, w.b, w.n_tokens, variant)
    _, gv = encode_both(xv, vcb, w.c, w.b, w.n_tokens, variant)
    H.check_codes(xk.numpy().reshape(-1, 1, 128), kcb.numpy(), gk.reshape(-1, 1, w.G), w.c, w.b, kres)
    H.check_codes(xv.numpy().reshape(-1, 1, 128), vcb.numpy(), gv.reshape(-1, 1, w.G), w.c, w.b, vres)
    out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [w.n_tokens], 128 ** -0.5, w.c, w.b, variant)
    H.check_attn(out, ref, "config 0")


@pytest.mark.parametrize("c,n_q,n_kv,lens", [
    (8, 4, 1, [1, 15, 16, 17, 0, 333]),          # GQA R=4, one-token, block edges, empty
    (8, 2, 2, [2049, 700]),                      # MHA, spans several splits
    (4, 2, 2, [257, 31]),
    (4, 4, 2, [1000, 1]),
    (2, 2, 2, [129, 64]),
    (2, 2, 1, [300]),
    (8, 8, 1, [90, 200]),                        # R = 8: two CTAs of four query heads per KV head
    (8, 3, 3, [50]),
    (8, 6, 2, [700, 2500]),                      # R = 3: three CTAs of one query head
    (8, 12, 2, [1300, 64]),                      # R = 6: three CTAs of two
    (4, 8, 2, [900, 33]),                        # 32 groups, R = 4: two CTAs of two
    (4, 3, 1, [515]),                            # 32 groups, R = 3
    (2, 4, 1, [2100, 17]),                       # 64 groups, R = 4: four CTAs of one
])
def test_attention_small_cases(c, n_q, n_kv, lens):
    b, D = 8, 128
    cap = max(max(lens), 1) + 5
    w = H.small_workload("t", 90 + c, c, b, len(lens), n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, len(lens), cap)
    xv = synth.layer_activations(w, 0, True, len(lens), cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(w.config, 0, len(lens), n_q)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    for variant in (1, 0):
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, D ** -0.5, c, b, variant)
        H.check_attn(out, ref, f"c={c} lens={lens} variant={variant}")
        for s, n in enumerate(lens):
            if n == 0:
                assert (out[s] == 0).all()
            if n == 1:      # a context of one token returns that token's V reconstruction
                vhat = oracle.dequant(vc_rm[s, :1].reshape(1, n_kv, -1), vcb.numpy(), c, b)[0]
                for hq in range(n_q):
                    np.testing.assert_allclose(out[s, hq], vhat[hq // (n_q // n_kv)], rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("c,b,head_dim,n_q,n_kv", [(1, 4, 64, 2, 2), (16, 8, 128, 2, 1), (8, 5, 64, 4, 2),
                                                   (4, 1, 32, 2, 2), (8, 8, 256, 2, 1), (2, 3, 16, 3, 3)])
def test_attention_generic_shapes(c, b, head_dim, n_q, n_kv):
    lens = [61, 7]
    cap = 64
    xk, xv, kcb, vcb, q = H.generic_case(100 + c * b, 2, cap, n_q, n_kv, head_dim, c, b)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, head_dim ** -0.5, c, b, 0)
    H.check_attn(out, ref, f"generic c={c} b={b} D={head_dim}")


def test_attention_peaked_and_flat_softmax():
    # a query aligned with one key (peaked weights) and a zero query (uniform weights)
    c, b, D, cap = 8, 8, 128, 1500
    w = H.small_workload("t", 77, c, b, 2, 1, 1, cap)
    xk = synth.layer_activations(w, 0, False, 2, cap)
    xv = synth.layer_activations(w, 0, True, 2, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    q = torch.zeros(2, 1, D, dtype=torch.float16)
    q[0, 0] = (4.0 * xk[0, 321, 0].float()).clamp(-60000, 60000).to(torch.float16)
    for variant in (1, 0):
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [cap, cap], 1.0, c, b, variant)
        H.check_attn(out, ref, f"peaked/flat variant={variant}")


@pytest.mark.parametrize("c,n_q,n_kv", [(8, 1, 1), (8, 4, 1), (8, 2, 1), (4, 1, 1), (4, 2, 1), (2, 1, 1), (8, 8, 1), (2, 2, 1)])
def test_weight_unit_is_coarsened_on_flat_and_on_rising_scores(c, n_q, n_kv):
    # Stress of the integer weight unit, for every tuned kernel shape.  Sequence 0: zero queries over
    # a long context (every weight equals the maximum, so the bins must coarsen their unit instead of
    # overflowing).  Sequence 1: tokens sorted by rising score of query head 0 with a large scale (the
    # running maximum keeps growing, and the other heads of a GQA group see different maxima).
    # Sequence 2: the same tokens in falling order (the first tokens dominate, the tail is tiny).
    b, D, cap = 8, 128, 20000
    w = H.small_workload("t", 78 + c + n_q, c, b, 3, n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, 3, cap)
    xv = synth.layer_activations(w, 0, True, 3, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    q = synth.queries(w.config, 0, 3, n_q)
    q[0] = 0
    q[2] = q[1]
    scale = 0.7
    khat = oracle.dequant(kc_rm[1].reshape(cap, n_kv, -1), kcb.numpy(), c, b)[:, 0]     # (cap, D)
    order = np.argsort(khat @ q[1, 0].double().numpy(), kind="stable")
    kc_rm[2], vc_rm[2] = kc_rm[1][order[::-1]], vc_rm[1][order[::-1]]
    kc_rm[1], vc_rm[1] = kc_rm[1][order], vc_rm[1][order]
    for variant in (1, 0):
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [cap, cap - 3, cap - 17], scale, c, b, variant)
        H.check_attn(out, ref, f"flat/rising/falling c={c} Hq={n_q} variant={variant}")
        for s_ in range(3):                      # per sequence too: a large row must not hide a small one
            H.check_attn(out[s_], ref[s_], f"flat/rising/falling seq {s_} c={c} Hq={n_q} variant={variant}")


def test_attention_multi_chunk_gqa_and_mha_long():
    # contexts long enough for several chunks per (sequence, KV head) and ragged ends
    for c, n_q, n_kv, lens in ((8, 4, 1, [9000, 4097]), (4, 1, 1, [5000]), (8, 2, 1, [6001]), (4, 2, 1, [4500]),
                               (2, 2, 2, [4100, 1025, 0])):
        b, D = 8, 128
        cap = max(lens) + 11
        w = H.small_workload("t", 120 + c + n_q, c, b, len(lens), n_q, n_kv, cap)
        xk = synth.layer_activations(w, 0, False, len(lens), cap)
        xv = synth.layer_activations(w, 0, True, len(lens), cap)
        kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
        q = synth.queries(w.config, 0, len(lens), n_q)
        kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
        vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, D ** -0.5, c, b, 0)
        H.check_attn(out, ref, f"long c={c} Hq={n_q} Hkv={n_kv}")


def test_attention_when_the_last_wave_of_items_is_spread_over_several_ctas():
    # 160 (sequence, KV head) items with one CTA per SM: the items beyond a multiple of the SM count
    # are spread over several CTAs each while the others take their whole context in one.  The spread
    # ones include a full-length sequence, a short one (its later parts are empty) and an empty one.
    c, b, D, n_q, n_kv = 8, 8, 128, 32, 8
    rng = np.random.default_rng(77)
    for lens_tail in ([8200, 100], [0, 8200]):
        lens = [int(v) for v in rng.integers(1, 8200, size=18)] + lens_tail
        n_seq, cap = len(lens), 8200
        kcb, vcb = (torch.from_numpy(rng.standard_normal((n_kv, D // c, 256, c)).astype(np.float32)) for _ in range(2))
        q = torch.from_numpy(rng.standard_normal((n_seq, n_q, D)).astype(np.float16))
        kc_rm = rng.integers(0, 256, size=(n_seq, cap, n_kv, D // c)).astype(np.int32)
        vc_rm = rng.integers(0, 256, size=(n_seq, cap, n_kv, D // c)).astype(np.int32)
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, D ** -0.5, c, b, 0)
        H.check_attn(out, ref, f"spread tail, lens of the last sequences {lens_tail}")
        for s_ in (n_seq - 2, n_seq - 1):
            H.check_attn(out[s_], ref[s_], f"spread tail, sequence {s_}")


def test_attention_with_codebooks_at_16_byte_offsets():
    # the tuned kernels read 8-channel centroids with 32-byte loads when both codebooks are 32-byte aligned
    # and with pairs of 16-byte loads otherwise: both paths must give the oracle's result
    c, b, D, n_q, n_kv, lens = 8, 8, 128, 4, 1, [3000, 77]
    cap = 3000
    w = H.small_workload("t", 131, c, b, 2, n_q, n_kv, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(w.config, 0, 2, n_q)
    rng = np.random.default_rng(4)
    kc_rm = rng.integers(0, 256, size=(2, cap, n_kv, D // c)).astype(np.int32)
    vc_rm = rng.integers(0, 256, size=(2, cap, n_kv, D // c)).astype(np.int32)
    kb = cq.cq_codes_from_rowmajor(torch.from_numpy(kc_rm.astype(np.uint8)).to(DEV), D, c, b)
    vb = cq.cq_codes_from_rowmajor(torch.from_numpy(vc_rm.astype(np.uint8)).to(DEV), D, c, b)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.asarray(lens, np.int32), D ** -0.5, c, b)
    def shifted(t):                      # same values, 16 bytes past a 256-byte aligned allocation
        buf = torch.empty(t.numel() + 4, dtype=torch.float32, device=DEV)
        v = buf[4:].view(t.shape)
        v.copy_(t)
        assert v.data_ptr() % 32 == 16
        return v
    for kd, vd in ((kcb.to(DEV), vcb.to(DEV)), (shifted(kcb), shifted(vcb)), (kcb.to(DEV), shifted(vcb))):
        out = cq.cq_decode_attn(q.to(DEV), kb, vb, kd, vd, sl, D ** -0.5, c, b, cap, variant=2).cpu().numpy()
        H.check_attn(out, ref, "codebook alignment")


def test_encode_codebooks_beyond_fp16_range_take_the_exact_path():
    # centroids too large for the fp16 term splits of the tensor-core path: the tuned kernel must
    # notice and recompute those groups exactly
    for c in (2, 4, 8):
        b, D, nh, n = 8, 128, 2, 48
        xk, _, kcb, _, _ = H.generic_case(500 + c, 1, n, nh, nh, D, c, b)
        kcb = kcb.clone()
        kcb[0, 1] *= 3.0e4                      # one group of head 0 far outside the range
        kcb[1, 0, 5] = 7.0e4                    # one centroid of another group
        for variant in (2, 0):
            _, rm = encode_both(xk, kcb, c, b, n, variant)
            H.check_codes(xk.numpy().reshape(-1, nh, D), kcb.numpy(), rm.reshape(-1, nh, D // c), c, b)


def test_attention_table_entries_beyond_fp16_range_are_prescaled():
    # |scale * <q_g, C>| far above 2^15: the table is rebuilt with a power-of-two prescale
    c, b, D, cap = 8, 8, 128, 300
    w = H.small_workload("t", 91, c, b, 2, 2, 1, cap)
    xk = synth.layer_activations(w, 0, False, 2, cap)
    xv = synth.layer_activations(w, 0, True, 2, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False) * 300.0, synth.layer_codebooks(w, 0, True)
    kc_rm, _ = H.oracle_encode_rowmajor((xk.float() * 300.0).clamp(-6e4, 6e4).to(torch.float16), kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    q = (synth.queries(91, 0, 2, 2).float() * 4).to(torch.float16)
    for variant in (1, 0):
        out, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [cap, 77], 1.0, c, b, variant)
        H.check_attn(out, ref, f"prescaled table variant={variant}")


def test_token_permutation_and_seq_len_padding_invariance():
    c, b, D, cap, n = 8, 8, 128, 640, 600
    w = H.small_workload("t", 55, c, b, 1, 4, 1, cap)
    xk = synth.layer_activations(w, 0, False, 1, cap)
    xv = synth.layer_activations(w, 0, True, 1, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(55, 0, 1, 4)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    base, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, [n], D ** -0.5, c, b, 0)
    H.check_attn(base, ref)
    perm = np.random.default_rng(1).permutation(n)
    kp, vp = kc_rm.copy(), vc_rm.copy()
    kp[0, :n], vp[0, :n] = kc_rm[0, perm], vc_rm[0, perm]
    kp[0, n:] = 255 - kp[0, n:]                       # garbage past seq_len must not matter
    out, _ = attn_both(q, kp, vp, kcb, vcb, [n], D ** -0.5, c, b, 0)
    np.testing.assert_allclose(out, base, rtol=0, atol=2e-5)


@pytest.mark.parametrize("packed,n_seq", [(False, 3), (True, 3), (True, 9), (False, 8)])
def test_decode_step_from_host_buffers(packed, n_seq):
    # packed: query, key and value back to back in one pinned block (they then travel in one copy)
    c, b, D, cap, n_q, n_kv = 8, 8, 128, 200, 4, 2
    w = H.small_workload("t", 66, c, b, n_seq, n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, n_seq, cap)
    xv = synth.layer_activations(w, 0, True, n_seq, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(66, 0, n_seq, n_q)
    lens = ([150, 0, 199] * 3)[:n_seq]         # tokens already cached; the step appends one more
    kbuf, _ = encode_both(xk, kcb, c, b, cap)
    vbuf, _ = encode_both(xv, vcb, c, b, cap)
    k_new = torch.stack([xk[s, 7] for s in range(n_seq)]).contiguous()      # (n_seq, n_kv, D)
    v_new = torch.stack([xv[s, 9] for s in range(n_seq)]).contiguous()
    ws = torch.empty(cq.cq_decode_step_host_workspace_bytes(n_seq, n_q, n_kv, D, c, b, cap), dtype=torch.uint8,
                     device=DEV)
    out_host = torch.empty(n_seq, n_q, D, dtype=torch.float32).pin_memory()
    if packed:
        block = torch.empty(q.numel() + k_new.numel() + v_new.numel(), dtype=torch.float16).pin_memory()
        hq = block[:q.numel()].view(q.shape)
        hk = block[q.numel():q.numel() + k_new.numel()].view(k_new.shape)
        hv = block[q.numel() + k_new.numel():].view(v_new.shape)
        hq.copy_(q); hk.copy_(k_new); hv.copy_(v_new)
    else:
        hq, hk, hv = q.pin_memory(), k_new.pin_memory(), v_new.pin_memory()
    cq.cq_decode_step_host(hq, hk, hv,
                           torch.tensor(lens, dtype=torch.int32), kbuf, vbuf, kcb.to(DEV), vcb.to(DEV),
                           D ** -0.5, c, b, cap, out_host, ws)
    # oracle: same cache with the new token written at position lens[s], context lens[s] + 1
    xk2, xv2 = xk.clone(), xv.clone()
    for s, n in enumerate(lens):
        xk2[s, n], xv2[s, n] = k_new[s], v_new[s]
    kc_rm, _ = H.oracle_encode_rowmajor(xk2, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv2, vcb, c, b)
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(),
                              np.asarray([n + 1 for n in lens], np.int32), D ** -0.5, c, b)
    H.check_attn(out_host.numpy(), ref, "host step")
    got_k = cq.cq_codes_to_rowmajor(kbuf, n_seq, cap, n_kv, D, c, b).cpu().numpy()
    for s, n in enumerate(lens):
        H.check_codes(k_new[s:s + 1].numpy(), kcb.numpy(), got_k[s, n][None], c, b)


def test_library_is_loaded_from_the_tree():
    import os
    assert os.path.samefile(os.path.dirname(cq.library_path()), os.path.dirname(cq.__file__))
    maps = open("/proc/self/maps").read()
    assert "libcq.so" in maps


@pytest.mark.parametrize("c,n_q,n_kv", [(8, 8, 2), (8, 2, 2), (4, 2, 1), (2, 1, 1)])
def test_repeated_calls_agree(c, n_q, n_kv):
    # Coarsening events depend on the order in which warps arrive, so the integer weight unit - and with it the
    # last bits of the output - may differ from run to run.  Twenty calls on the same inputs: the spread of
    # every output element is reported and bounded (2e-6 absolute is a thousandth of the max-abs tolerance).
    lens = [5000, 1234, 4096, 77]
    cap = 5000
    w = H.small_workload("repeat", 0, c, 8, len(lens), n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, len(lens), cap)
    xv = synth.layer_activations(w, 0, True, len(lens), cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False).to(DEV), synth.layer_codebooks(w, 0, True).to(DEV)
    kb = torch.zeros(cq.cq_codes_bytes(len(lens), cap, n_kv, 128, c, 8), dtype=torch.uint8, device=DEV)
    vb = torch.zeros_like(kb)
    cq.cq_encode_kv(xk.to(DEV), xv.to(DEV), kcb, vcb, c, 8, kb, vb, cap)
    q = synth.queries(0, 0, len(lens), n_q).to(DEV)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    outs = torch.stack([cq.cq_decode_attn(q, kb, vb, kcb, vcb, sl, 128 ** -0.5, c, 8, cap).clone() for _ in range(20)])
    spread = float((outs.max(dim=0).values - outs.min(dim=0).values).max().item())
    print(f"c={c} R={n_q // n_kv}: largest spread over 20 calls {spread:.3e}")
    assert spread <= 2e-6


@pytest.mark.parametrize("n_q,n_kv", [(4, 1), (8, 1), (16, 2)])
def test_both_tuned_kernels_for_four_heads_per_kv_head(n_q, n_kv):
    # CQ-8c8b with a multiple of four query heads per KV head has two tuned kernels: the one with two query heads
    # per table word (variant 2, what variant 0 picks) and the one with a table word per query head (variant 3).
    lens = [3000, 17, 2049, 0, 512]
    cap = 3000
    w = H.small_workload("two_kernels", 0, 8, 8, len(lens), n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, len(lens), cap)
    xv = synth.layer_activations(w, 0, True, len(lens), cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, 8, 8)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, 8, 8)
    q = synth.queries(0, 0, len(lens), n_q)
    for variant in (2, 3):
        got, ref = attn_both(q, kc_rm, vc_rm, kcb, vcb, lens, 128 ** -0.5, 8, 8, variant)
        for s_ in range(len(lens)):
            H.check_attn(got[s_], ref[s_], f"variant {variant} seq {s_}")
