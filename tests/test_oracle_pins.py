"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible slip in the oracle (wrong group or head index, transposed codebook,
dropped scale, wrong GQA mapping, missing normalisation) breaks it.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(20240503)


def rand_case(n_vec, n_heads, D, c, b, scale_x=1.0):
    x = (scale_x * rng.standard_normal((n_vec, n_heads, D))).astype(np.float16)
    cb = rng.standard_normal((n_heads, D // c, 1 << b, c)).astype(np.float32)
    return x, cb


# ----------------------------------------------------------------------------- encode

def test_fp16_widening_is_exact():
    # K = 1 centroid at 0, c = 1: distance is x^2, so every finite fp16 bit pattern
    # must come back as numpy's own widening squared.
    bits = np.arange(65536, dtype=np.uint16)
    vals = bits.view(np.float16).astype(np.float64)
    keep = np.isfinite(vals)
    x = bits[keep].reshape(-1, 1, 1)
    cb = np.zeros((1, 1, 1, 1), dtype=np.float32)
    codes, d1, _ = oracle.encode(x, cb, 1, 0)
    assert (codes == 0).all()
    assert np.array_equal(d1.ravel(), vals[keep] ** 2)


def test_hand_worked_scalar_and_pair_cases():
    # c = 1, centroids {0, 10}: 4 -> 0, 6 -> 1, 5 is an exact tie -> lowest index.
    x = np.array([4.0, 6.0, 5.0, -3.0, 11.0], dtype=np.float16).reshape(5, 1, 1)
    cb = np.array([0.0, 10.0], dtype=np.float32).reshape(1, 1, 2, 1)
    codes, d1, d2 = oracle.encode(x, cb, 1, 1)
    assert codes.ravel().tolist() == [0, 1, 0, 0, 1]
    assert d1.ravel().tolist() == [16.0, 16.0, 25.0, 9.0, 1.0]
    assert d2.ravel().tolist() == [36.0, 36.0, 25.0, 169.0, 121.0]
    # c = 2, b = 2, one vector of two groups with different codebooks per group.
    # group 0 = (1, 1): centroids (0,0) d=2, (2,2) d=2, (1,2) d=1, (3,1) d=4 -> 2
    # group 1 = (-2, 0): centroids (0,0) d=4, (-2,1) d=1, (-3,0) d=1, (5,5) -> tie 1/2 -> 1
    x = np.array([1, 1, -2, 0], dtype=np.float16).reshape(1, 1, 4)
    cb = np.array([[[0, 0], [2, 2], [1, 2], [3, 1]],
                   [[0, 0], [-2, 1], [-3, 0], [5, 5]]], dtype=np.float32).reshape(1, 2, 4, 2)
    codes, d1, d2 = oracle.encode(x, cb, 2, 2)
    assert codes.ravel().tolist() == [2, 1]
    assert d1.ravel().tolist() == [1.0, 1.0]
    assert d2.ravel().tolist() == [2.0, 1.0]


@pytest.mark.parametrize("c,b", [(1, 1), (2, 2), (4, 3), (8, 2), (2, 3)])
def test_brute_force_python_loops(c, b):
    # Integer-valued tiny inputs, distances by pure-Python integer arithmetic.
    D, n_vec, n_heads = 8, 6, 2
    x = rng.integers(-4, 5, size=(n_vec, n_heads, D)).astype(np.float16)
    cb = rng.integers(-4, 5, size=(n_heads, D // c, 1 << b, c)).astype(np.float32)
    codes, d1, d2 = oracle.encode(x, cb, c, b)
    for v, h, g in itertools.product(range(n_vec), range(n_heads), range(D // c)):
        ds = []
        for j in range(1 << b):
            ds.append(sum((int(x[v, h, g * c + i]) - int(cb[h, g, j, i])) ** 2 for i in range(c)))
        best = min(ds)
        assert codes[v, h, g] == ds.index(best)          # first occurrence
        assert d1[v, h, g] == best
        assert d2[v, h, g] == sorted(ds)[1]


@pytest.mark.parametrize("c,b", [(2, 8), (4, 8), (8, 8), (8, 5)])
def test_codebook_contains_inputs_gives_zero_error(c, b):
    # Every input group is one of its group's centroids: distance exactly 0,
    # code = lowest index holding that centroid, reconstruction = input.
    D, n_heads, K = 32, 3, 1 << b
    cb = rng.standard_normal((n_heads, D // c, K, c)).astype(np.float16).astype(np.float32)
    cb[:, :, K - 1, :] = cb[:, :, 3, :]                   # duplicate: index 3 must win over K-1
    pick = rng.integers(0, K, size=(50, n_heads, D // c))
    x = np.empty((50, n_heads, D), dtype=np.float16)
    for v, h, g in itertools.product(range(50), range(n_heads), range(D // c)):
        x[v, h, g * c:(g + 1) * c] = cb[h, g, pick[v, h, g]]
    codes, d1, _ = oracle.encode(x, cb, c, b)
    want = np.where(pick == K - 1, 3, pick)
    assert np.array_equal(codes, want)
    assert (d1 == 0).all()
    assert np.array_equal(oracle.dequant(codes, cb, c, b), x.astype(np.float64))


def test_c1_reduces_to_scalar_bucketing():
    # With one channel per group CQ is channel-wise non-uniform quantisation
    # (Section 2.3): nearest scalar centroid = bucket between sorted midpoints.
    D, b = 16, 4
    x = rng.standard_normal((200, 1, D)).astype(np.float16)
    cb = rng.standard_normal((1, D, 1 << b, 1)).astype(np.float32)
    codes, _, _ = oracle.encode(x, cb, 1, b)
    for ch in range(D):
        cent = cb[0, ch, :, 0].astype(np.float64)
        order = np.argsort(cent, kind="stable")
        mids = (cent[order][1:] + cent[order][:-1]) / 2
        want = order[np.searchsorted(mids, x[:, 0, ch].astype(np.float64), side="left")]
        assert np.array_equal(codes[:, 0, ch], want)


@pytest.mark.parametrize("c,b", [(2, 8), (4, 6), (8, 8), (8, 10), (4, 9)])
def test_matches_torch_cdist_argmin(c, b):
    D, n_heads = 64, 3
    x, cb = rand_case(40, n_heads, D, c, b)
    codes, d1, d2 = oracle.encode(x, cb, c, b)
    xt = torch.from_numpy(x.astype(np.float64))
    for h in range(n_heads):
        for g in range(D // c):
            dist = torch.cdist(xt[:, h, g * c:(g + 1) * c], torch.from_numpy(cb[h, g].astype(np.float64))) ** 2
            assert np.array_equal(codes[:, h, g], dist.argmin(dim=1).numpy())
            top2 = dist.topk(2, dim=1, largest=False).values.numpy()
            np.testing.assert_allclose(d1[:, h, g], top2[:, 0], rtol=1e-9)   # cdist takes a sqrt
            np.testing.assert_allclose(d2[:, h, g], top2[:, 1], rtol=1e-9)


def test_single_code_change_never_lowers_error():
    # Objective of CQ(.) in Eq. 5: nearest-centroid assignment minimises ||A - CQ(A)||_F^2.
    D, c, b = 32, 4, 6
    x, cb = rand_case(30, 2, D, c, b)
    codes, _, _ = oracle.encode(x, cb, c, b)
    base = ((oracle.dequant(codes, cb, c, b) - x.astype(np.float64)) ** 2).sum()
    for _ in range(200):
        alt = codes.copy()
        v, h, g = rng.integers(30), rng.integers(2), rng.integers(D // c)
        alt[v, h, g] = rng.integers(1 << b)
        err = ((oracle.dequant(alt, cb, c, b) - x.astype(np.float64)) ** 2).sum()
        assert err >= base - 1e-9
    dist = oracle.code_distance(x, cb, codes, c, b)
    np.testing.assert_allclose(dist.sum(), base, rtol=1e-12)


def test_sizes_match_paper_tables():
    for line in open(os.path.join(GOLDEN, "table4_centroid_params.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, layers, heads, hd, bits, printed = line.split()
        n = int(layers) * 2 * int(heads) * int(hd) * (1 << int(bits))
        assert round(n / 1e6, 2) == float(printed)
        for c in (2, 4, 8):   # the count does not depend on the coupling c
            cb_shape = (int(heads), int(hd) // c, 1 << int(bits), c)
            assert int(layers) * 2 * int(np.prod(cb_shape)) == n
    for line in open(os.path.join(GOLDEN, "table1_bits_per_fpn.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, c, b, printed = line.split()
        assert int(b) / int(c) == float(printed)


# ----------------------------------------------------------------------------- attention

def attn_case(n_seq, Hq, Hkv, D, c, b, max_tokens, lens=None):
    q = rng.standard_normal((n_seq, Hq, D)).astype(np.float16)
    kc = rng.integers(0, 1 << b, size=(n_seq, max_tokens, Hkv, D // c)).astype(np.int32)
    vc = rng.integers(0, 1 << b, size=(n_seq, max_tokens, Hkv, D // c)).astype(np.int32)
    kcb = rng.standard_normal((Hkv, D // c, 1 << b, c)).astype(np.float32)
    vcb = rng.standard_normal((Hkv, D // c, 1 << b, c)).astype(np.float32)
    sl = np.full(n_seq, max_tokens, dtype=np.int32) if lens is None else np.asarray(lens, dtype=np.int32)
    return q, kc, vc, kcb, vcb, sl


def torch_dense(q, kc, vc, kcb, vcb, sl, scale, c, b):
    """Eq. 1 with library routines: gather, matmul, torch.softmax, all fp64."""
    n_seq, Hq, D = q.shape
    Hkv = kc.shape[2]
    G = D // c
    R = Hq // Hkv
    out = np.zeros((n_seq, Hq, D))
    for s in range(n_seq):
        n = int(sl[s])
        if n == 0:
            continue
        for hq in range(Hq):
            h = hq // R
            gi = torch.arange(G)
            K = torch.from_numpy(kcb[h].astype(np.float64))[gi[None, :], torch.from_numpy(kc[s, :n, h].astype(np.int64))].reshape(n, D)
            V = torch.from_numpy(vcb[h].astype(np.float64))[gi[None, :], torch.from_numpy(vc[s, :n, h].astype(np.int64))].reshape(n, D)
            p = torch.softmax(scale * (K @ torch.from_numpy(q[s, hq].astype(np.float64))), dim=0)
            out[s, hq] = (p[None, :] @ V).numpy()[0]
    return out


@pytest.mark.parametrize("c,b,Hq,Hkv", [(8, 8, 4, 2), (4, 8, 2, 2), (2, 5, 6, 2), (8, 10, 2, 1)])
def test_dense_matches_torch_softmax(c, b, Hq, Hkv):
    D = 32
    args = attn_case(3, Hq, Hkv, D, c, b, 37, lens=[37, 5, 0])
    got = oracle.decode_dense(*args, 0.31, c, b)
    want = torch_dense(*args, 0.31, c, b)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)
    assert (got[2] == 0).all()                     # empty context -> zero row


@pytest.mark.parametrize("n_chunks", [1, 2, 7, 53])
def test_lut_form_equals_dense_form_for_any_chunking(n_chunks):
    args = attn_case(2, 4, 2, 64, 8, 8, 53, lens=[53, 20])
    dense = oracle.decode_dense(*args, 1 / np.sqrt(64), 8, 8)
    lut = oracle.decode_lut(*args, 1 / np.sqrt(64), 8, 8, n_chunks=n_chunks)
    np.testing.assert_allclose(lut, dense, rtol=1e-12, atol=1e-14)


def test_lut_sum_equals_scaled_dot_with_reconstruction():
    # sum_g LUT_g[code_g] = scale <q, Khat>, checked through a context of two tokens:
    # out = sigma(s0 - s1) V0 + (1 - sigma) V1 with s from an independent numpy dot.
    D, c, b = 16, 4, 3
    q, kc, vc, kcb, vcb, sl = attn_case(1, 1, 1, D, c, b, 2)
    scale = 0.7
    khat = oracle.dequant(kc[0], kcb, c, b)[:, 0]     # (2, D)
    vhat = oracle.dequant(vc[0], vcb, c, b)[:, 0]
    s = scale * khat @ q[0, 0].astype(np.float64)
    w0 = 1 / (1 + np.exp(s[1] - s[0]))
    want = w0 * vhat[0] + (1 - w0) * vhat[1]
    for fn in (lambda: oracle.decode_dense(q, kc, vc, kcb, vcb, sl, scale, c, b),
               lambda: oracle.decode_lut(q, kc, vc, kcb, vcb, sl, scale, c, b, n_chunks=2)):
        np.testing.assert_allclose(fn()[0, 0], want, rtol=1e-12, atol=1e-14)


def test_one_token_context_returns_its_value_reconstruction():
    D, c, b = 128, 8, 8
    q, kc, vc, kcb, vcb, _ = attn_case(3, 4, 2, D, c, b, 5)
    sl = np.ones(3, dtype=np.int32)
    out = oracle.decode_dense(q, kc, vc, kcb, vcb, sl, 0.088, c, b)
    for s in range(3):
        vhat = oracle.dequant(vc[s, :1], vcb, c, b)[0]          # (Hkv, D)
        for hq in range(4):
            assert np.array_equal(out[s, hq], vhat[hq // 2])


def test_zero_query_gives_mean_and_score_shift_is_invisible():
    D, c, b = 32, 4, 4
    q, kc, vc, kcb, vcb, sl = attn_case(1, 2, 1, D, c, b, 19)
    kcb = np.round(kcb * 64) / 64                       # so that the shift below is exact in fp32
    out0 = oracle.decode_dense(np.zeros_like(q), kc, vc, kcb, vcb, sl, 0.5, c, b)
    vhat = oracle.dequant(vc[0, :, :, :], vcb, c, b)[:, 0]
    np.testing.assert_allclose(out0[0, 0], vhat.mean(axis=0), rtol=1e-12, atol=1e-14)
    base = oracle.decode_dense(q, kc, vc, kcb, vcb, sl, 0.5, c, b)
    shifted = kcb.copy()
    shifted[0, 3] += np.array([0.5, -1.25, 2.0, 0.75], dtype=np.float32)   # same shift for every centroid of group 3
    np.testing.assert_allclose(oracle.decode_dense(q, kc, vc, shifted, vcb, sl, 0.5, c, b), base,
                               rtol=1e-9, atol=1e-12)


def test_token_permutation_and_gqa_replication():
    D, c, b = 32, 8, 6
    q, kc, vc, kcb, vcb, sl = attn_case(2, 4, 2, D, c, b, 23, lens=[23, 11])
    base = oracle.decode_dense(q, kc, vc, kcb, vcb, sl, 0.2, c, b)
    kp, vp = kc.copy(), vc.copy()
    for s in range(2):
        perm = rng.permutation(int(sl[s]))
        kp[s, :sl[s]] = kc[s, perm]
        vp[s, :sl[s]] = vc[s, perm]
    np.testing.assert_allclose(oracle.decode_dense(q, kp, vp, kcb, vcb, sl, 0.2, c, b), base,
                               rtol=1e-11, atol=1e-13)
    # GQA with R = 2 equals MHA with every KV head (codes and codebooks) repeated twice.
    rep = lambda a, ax: np.repeat(a, 2, axis=ax)
    mha = oracle.decode_dense(q, rep(kc, 2), rep(vc, 2), rep(kcb, 0), rep(vcb, 0), sl, 0.2, c, b)
    assert np.array_equal(mha, base)
    # tokens past seq_len are never read
    kc2 = kc.copy()
    kc2[1, 11:] = (kc2[1, 11:] + 1) % (1 << b)
    assert np.array_equal(oracle.decode_dense(q, kc2, vc, kcb, vcb, sl, 0.2, c, b), base)


def test_scale_is_applied_to_scores_only():
    D, c, b = 16, 2, 3
    q, kc, vc, kcb, vcb, sl = attn_case(1, 1, 1, D, c, b, 9)
    a = oracle.decode_dense(q, kc, vc, kcb, vcb, sl, 0.25, c, b)
    b2 = oracle.decode_dense(q, kc, vc, (0.25 * kcb.astype(np.float64)).astype(np.float32), vcb, sl, 1.0, c, b)
    np.testing.assert_allclose(a, b2, rtol=1e-6)      # 0.25 is a power of two: kcb scaling is exact
    assert np.abs(a - oracle.decode_dense(q, kc, vc, kcb, vcb, sl, 1.0, c, b)).max() > 1e-3


# ----------------------------------------------------------------------------- causal attention of a run of new tokens

def prefill_case(n_seq, n_q, Hq, Hkv, D, c, b, max_tokens, lens):
    _, kc, vc, kcb, vcb, sl = attn_case(n_seq, Hq, Hkv, D, c, b, max_tokens, lens=lens)
    q = rng.standard_normal((n_seq, n_q, Hq, D)).astype(np.float16)
    return q, kc, vc, kcb, vcb, sl


@pytest.mark.parametrize("c,b,Hq,Hkv", [(8, 8, 4, 2), (4, 6, 2, 2), (2, 5, 6, 2)])
def test_prefill_matches_torch_masked_softmax(c, b, Hq, Hkv):
    # Eq. 1 for all queries at once with library routines: one score matrix, a causal mask, torch.softmax.
    D, n_q = 32, 7
    q, kc, vc, kcb, vcb, sl = prefill_case(3, n_q, Hq, Hkv, D, c, b, 29, lens=[29, 11, 4])
    got = oracle.prefill_dense(q, kc, vc, kcb, vcb, sl, 0.23, c, b)
    G, R = D // c, Hq // Hkv
    gi = torch.arange(G)
    for s in range(3):
        n = int(sl[s])
        for hq in range(Hq):
            h = hq // R
            K = torch.from_numpy(kcb[h].astype(np.float64))[gi[None, :], torch.from_numpy(kc[s, :n, h].astype(np.int64))].reshape(n, D)
            V = torch.from_numpy(vcb[h].astype(np.float64))[gi[None, :], torch.from_numpy(vc[s, :n, h].astype(np.int64))].reshape(n, D)
            Q = torch.from_numpy(q[s, :, hq].astype(np.float64))                       # (n_q, D)
            S = 0.23 * (Q @ K.T)                                                         # (n_q, n)
            pos = n - n_q + torch.arange(n_q)                                            # position of query i
            mask = torch.arange(n)[None, :] > pos[:, None]
            S = S.masked_fill(mask, float("-inf"))
            want = torch.zeros(n_q, D, dtype=torch.float64)
            ok = pos >= 0
            want[ok] = torch.softmax(S[ok], dim=1) @ V
            np.testing.assert_allclose(got[s, :, hq], want.numpy(), rtol=1e-11, atol=1e-13)
    assert (got[2, :3] == 0).all()          # sequence 2 caches 4 tokens for 7 queries: the first three have no position


def test_prefill_row_equals_single_query_attention_at_that_length():
    # Row i is Eq. 1 for one query over the first pos_i + 1 tokens: the decode form, which has its own pins.
    D, c, b, n_q = 32, 8, 6, 5
    q, kc, vc, kcb, vcb, sl = prefill_case(2, n_q, 4, 2, D, c, b, 23, lens=[23, 9])
    got = oracle.prefill_dense(q, kc, vc, kcb, vcb, sl, 0.2, c, b)
    for i in range(n_q):
        one = oracle.decode_dense(np.ascontiguousarray(q[:, i]), kc, vc, kcb, vcb, sl - n_q + i + 1, 0.2, c, b)
        assert np.array_equal(got[:, i], one)


def test_prefill_hand_worked_and_first_token():
    # A prompt that is the whole cache: query 0 sees only token 0 and returns its value reconstruction
    # exactly; query 1 sees two tokens: out = sigma(s0 - s1) V0 + (1 - sigma) V1.
    D, c, b = 16, 4, 3
    q, kc, vc, kcb, vcb, sl = prefill_case(1, 3, 1, 1, D, c, b, 3, lens=[3])
    scale = 0.6
    got = oracle.prefill_dense(q, kc, vc, kcb, vcb, sl, scale, c, b)
    khat = oracle.dequant(kc[0], kcb, c, b)[:, 0]
    vhat = oracle.dequant(vc[0], vcb, c, b)[:, 0]
    assert np.array_equal(got[0, 0, 0], vhat[0])
    s = scale * khat[:2] @ q[0, 1, 0].astype(np.float64)
    w0 = 1 / (1 + np.exp(s[1] - s[0]))
    np.testing.assert_allclose(got[0, 1, 0], w0 * vhat[0] + (1 - w0) * vhat[1], rtol=1e-12, atol=1e-14)


def test_prefill_sees_no_future_token_and_no_order_in_the_past():
    D, c, b, n_q = 32, 4, 5, 6
    q, kc, vc, kcb, vcb, sl = prefill_case(1, n_q, 2, 1, D, c, b, 20, lens=[17])
    base = oracle.prefill_dense(q, kc, vc, kcb, vcb, sl, 0.3, c, b)
    # changing the codes of new token j changes rows j.. only; tokens past seq_len are never read
    j = 3
    k2, v2 = kc.copy(), vc.copy()
    t = 17 - n_q + j
    k2[0, t] = (k2[0, t] + 1) % (1 << b)
    v2[0, t] = (v2[0, t] + 3) % (1 << b)
    k2[0, 17:] = (k2[0, 17:] + 1) % (1 << b)
    got = oracle.prefill_dense(q, k2, v2, kcb, vcb, sl, 0.3, c, b)
    assert np.array_equal(got[0, :j], base[0, :j])
    assert all(np.abs(got[0, i] - base[0, i]).max() > 1e-9 for i in range(j, n_q))
    # permuting the tokens cached before the first query leaves every row unchanged
    perm = rng.permutation(17 - n_q)
    kp, vp = kc.copy(), vc.copy()
    kp[0, :17 - n_q] = kc[0, perm]
    vp[0, :17 - n_q] = vc[0, perm]
    np.testing.assert_allclose(oracle.prefill_dense(q, kp, vp, kcb, vcb, sl, 0.3, c, b), base, rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------- centroid learning

def _golden_kmeans():
    rows = []
    for line in open(os.path.join(GOLDEN, "kmeans_hand_worked.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, *cols = [f.strip() for f in line.split("|")]
        rows.append((head.split(), [np.array(col.split(), dtype=np.float64) for col in cols]))
    return rows


def _as_problem(points):
    """1-D points as a (n, 1 head, D = 1) fp16 array: one head, one group of one channel."""
    return np.asarray(points, dtype=np.float16).reshape(-1, 1, 1)


# ----------------------------------------------------------------------------- keys coded before RoPE

def rope_tables(max_tokens, P, base=10000.0, offset=0):
    """cos / sin of t * base^(-i/P) as models cache them (fp32), positions offset .. offset + max_tokens - 1."""
    t = np.arange(offset, offset + max_tokens, dtype=np.float64)[:, None]
    ang = t * base ** (-np.arange(P, dtype=np.float64) / P)[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def test_rope_identity_tables_give_the_plain_attention():
    args = attn_case(2, 4, 2, 32, 8, 8, 29, lens=[29, 6])
    cs, sn = np.ones((29, 16), np.float32), np.zeros((29, 16), np.float32)
    for pairing in (0, 1):
        got = oracle.decode_dense_rope(*args, cs, sn, 0.4, 8, 8, pairing)
        assert np.array_equal(got, oracle.decode_dense(*args, 0.4, 8, 8))


def test_rope_hand_worked_quarter_turns():
    # D = 2, one pair, c = 1 (two groups of one channel), two code values per group: centroids {1, 3} and {2, 5}.
    # Token 0 = (1, 2) at angle 0, token 1 = (3, 5) turned by 90 degrees = (-5, 3).  q = (1, 1), scale 1:
    # scores (3, -2); values are the V centroids (10, 20) and (30, 40).
    q = np.array([[[1.0, 1.0]]], np.float16)
    kcb = np.array([[[[1.0], [3.0]], [[2.0], [5.0]]]], np.float32)          # (1 head, 2 groups, 2 codes, c = 1)
    vcb = np.array([[[[10.0], [30.0]], [[20.0], [40.0]]]], np.float32)
    codes = np.array([[[[0, 0]], [[1, 1]]]], np.int32)                        # (1 seq, 2 tokens, 1 head, 2 groups)
    cs = np.array([[1.0], [0.0]], np.float32)
    sn = np.array([[0.0], [1.0]], np.float32)
    got = oracle.decode_dense_rope(q, codes, codes, kcb, vcb, [2], cs, sn, 1.0, 1, 1, 0)
    p0 = 1.0 / (1.0 + np.exp(-5.0))
    np.testing.assert_allclose(got[0, 0], [10 * p0 + 30 * (1 - p0), 20 * p0 + 40 * (1 - p0)], rtol=1e-14)
    # with D = 2 both pairings name the same pair
    assert np.array_equal(got, oracle.decode_dense_rope(q, codes, codes, kcb, vcb, [2], cs, sn, 1.0, 1, 1, 1))


@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_matches_torch_rotation(pairing):
    D, c, b, n = 32, 4, 6, 41
    q, kc, vc, kcb, vcb, sl = attn_case(2, 2, 1, D, c, b, n, lens=[41, 17])
    cs, sn = rope_tables(n, D // 2)
    got = oracle.decode_dense_rope(q, kc, vc, kcb, vcb, sl, cs, sn, 0.3, c, b, pairing)
    G = D // c
    gi = torch.arange(G)
    for s in range(2):
        m = int(sl[s])
        K = torch.from_numpy(kcb[0].astype(np.float64))[gi[None, :], torch.from_numpy(kc[s, :m, 0].astype(np.int64))].reshape(m, D)
        V = torch.from_numpy(vcb[0].astype(np.float64))[gi[None, :], torch.from_numpy(vc[s, :m, 0].astype(np.int64))].reshape(m, D)
        C, S = torch.from_numpy(cs[:m].astype(np.float64)), torch.from_numpy(sn[:m].astype(np.float64))
        if pairing == 0:      # rotate_half: x * [cos, cos] + [-x2, x1] * [sin, sin]
            Kr = K * torch.cat([C, C], 1) + torch.cat([-K[:, D // 2:], K[:, :D // 2]], 1) * torch.cat([S, S], 1)
        else:                 # complex multiplication of (x_2i + i x_2i+1) by e^{i angle}
            z = torch.view_as_complex(K.reshape(m, D // 2, 2).contiguous()) * torch.complex(C, S)
            Kr = torch.view_as_real(z).reshape(m, D)
        for hq in range(2):
            p = torch.softmax(0.3 * (Kr @ torch.from_numpy(q[s, hq].astype(np.float64))), dim=0)
            np.testing.assert_allclose(got[s, hq], (p[None, :] @ V).numpy()[0], rtol=1e-11, atol=1e-13)


def test_rope_scores_depend_on_relative_position_only():
    # Quarter-turn angles are exact in fp32 (cos, sin in {0, 1, -1}): pair i turns by (i % 4) quarter turns per
    # position.  Turning the query by the angles of position Delta and shifting every key position by Delta
    # leaves every score, hence the output, unchanged.
    D, c, b, n, delta = 16, 4, 5, 23, 5
    q, kc, vc, kcb, vcb, sl = attn_case(1, 1, 1, D, c, b, n)
    P = D // 2
    def tables(offset):
        k = ((np.arange(offset, offset + n)[:, None]) * (np.arange(P)[None, :] % 4)) % 4
        return np.array([1, 0, -1, 0], np.float32)[k], np.array([0, 1, 0, -1], np.float32)[k]
    base = oracle.decode_dense_rope(q, kc, vc, kcb, vcb, sl, *tables(0), 0.5, c, b, 0)
    # the query turned by delta positions (exact: a signed permutation of its channels)
    cd, sd = tables(delta)[0][0], tables(delta)[1][0]
    qf = q.astype(np.float64)[0, 0]
    qr = np.concatenate([qf[:P] * cd - qf[P:] * sd, qf[P:] * cd + qf[:P] * sd]).astype(np.float16)[None, None]
    shifted = oracle.decode_dense_rope(qr, kc, vc, kcb, vcb, sl, *tables(delta), 0.5, c, b, 0)
    np.testing.assert_allclose(shifted, base, rtol=1e-12, atol=1e-14)


def test_rope_pairings_differ_by_a_channel_permutation():
    # interleaved pairs (2i, 2i+1) of permuted inputs = half-split pairs (i, i + D/2) of the original ones
    D, b, n = 16, 4, 19
    q, kc, vc, kcb, vcb, sl = attn_case(1, 2, 1, D, 1, b, n)               # c = 1: any channel order is a valid grouping
    cs, sn = rope_tables(n, D // 2)
    perm = np.empty(D, np.int64)
    perm[0::2], perm[1::2] = np.arange(D // 2), np.arange(D // 2) + D // 2  # new channel 2i <- i, 2i+1 <- i + D/2
    half = oracle.decode_dense_rope(q, kc, vc, kcb, vcb, sl, cs, sn, 0.7, 1, b, 0)
    inter = oracle.decode_dense_rope(q[..., perm], kc[..., perm], vc, kcb[:, perm], vcb, sl, cs, sn, 0.7, 1, b, 1)
    np.testing.assert_allclose(inter, half, rtol=1e-12, atol=1e-14)


def test_rope_single_token_returns_its_value():
    q, kc, vc, kcb, vcb, _ = attn_case(1, 1, 1, 16, 4, 4, 9)
    cs, sn = rope_tables(9, 8)
    got = oracle.decode_dense_rope(q, kc, vc, kcb, vcb, [1], cs, sn, 1.0, 4, 4, 0)
    np.testing.assert_allclose(got[0, 0], oracle.dequant(vc[0, :1], vcb, 4, 4)[0, 0], rtol=1e-15)


def test_lloyd_step_hand_worked_cases():
    n_cases = 0
    for (kind, name), cols in _golden_kmeans():
        if kind != "lloyd":
            continue
        pts, w, cin, cout, obj = cols
        K = len(cin)
        b = int(np.log2(K)) if K & (K - 1) == 0 else None
        if b is None:                 # pad a 3-centroid case to 4 with a far copy that stays empty
            cin = np.append(cin, 1e4)
            cout = np.append(cout, 1e4)
            b = 2
        new, codes, o = oracle.lloyd_step(_as_problem(pts), w.reshape(-1, 1, 1).astype(np.float32),
                                          cin.reshape(1, 1, -1, 1).astype(np.float32), 1, b)
        np.testing.assert_allclose(new.reshape(-1), cout, rtol=0, atol=1e-6, err_msg=name)
        assert abs(o[0, 0] - obj[0]) < 1e-9, name
        n_cases += 1
    assert n_cases == 4


def test_kmeanspp_hand_worked_cases():
    n_cases = 0
    for (kind, name), cols in _golden_kmeans():
        if kind != "kmeanspp":
            continue
        pts, w, u, chosen = cols
        K = 4                          # 3 draws checked; a fourth centre pads to a power of two
        uu = np.append(u, 0.5).reshape(1, 1, K)
        cb, ch = oracle.kmeanspp_init(_as_problem(pts), w.reshape(-1, 1, 1).astype(np.float32), uu, 1, 2)
        assert ch[0, 0, :3].tolist() == chosen.astype(int).tolist(), name
        np.testing.assert_array_equal(cb[0, 0, :3, 0], pts[chosen.astype(int)])
        n_cases += 1
    assert n_cases == 3


def test_lloyd_step_matches_sklearn_one_iteration():
    from sklearn.cluster import KMeans
    r = np.random.default_rng(7)
    for c, b, weighted in ((2, 3, False), (4, 4, True), (8, 3, True)):
        n, K = 600, 1 << b
        x = r.standard_normal((n, 1, c)).astype(np.float16)
        w = (r.random((n, 1, 1)) + 0.1).astype(np.float32) if weighted else None
        init = x[r.choice(n, K, replace=False), 0].astype(np.float32)            # members guaranteed: no empty cluster
        new, codes, obj = oracle.lloyd_step(x, w, init.reshape(1, 1, K, c), c, b)
        km = KMeans(n_clusters=K, init=init.astype(np.float64), n_init=1, max_iter=1, tol=0.0, algorithm="lloyd")
        km.fit(x[:, 0].astype(np.float64), sample_weight=None if w is None else w[:, 0, 0].astype(np.float64))
        np.testing.assert_allclose(new[0, 0], km.cluster_centers_, rtol=1e-6, atol=1e-6)


def test_lloyd_objective_never_increases_and_means_are_optimal():
    r = np.random.default_rng(8)
    c, b, n = 4, 4, 800
    x = r.standard_normal((n, 2, 8)).astype(np.float16)
    w = r.random((n, 2, 2)).astype(np.float32)
    cb, _ = oracle.kmeanspp_init(x, w, r.random((2, 2, 16)), c, b)
    last = None
    for _ in range(6):
        new, codes, obj = oracle.lloyd_step(x, w, cb, c, b)
        if last is not None:
            assert (obj <= last * (1 + 1e-12)).all()
        last = obj
        # for the fixed assignment, moving any centroid away from the weighted mean raises the objective
        xf = x.astype(np.float64)
        for h, g in ((0, 0), (1, 1)):
            grp = xf[:, h, g * c:(g + 1) * c]
            cost = lambda cc: float((w[:, h, g] * ((grp - cc[codes[:, h, g]]) ** 2).sum(1)).sum())
            base = cost(new[h, g].astype(np.float64))
            for _t in range(5):
                pert = new[h, g].astype(np.float64).copy()
                pert[r.integers(16), r.integers(c)] += r.choice([-1, 1]) * 0.05
                assert cost(pert) >= base - 1e-9
        cb = new


def test_kmeanspp_picks_every_point_once_when_points_equal_centres():
    r = np.random.default_rng(9)
    c, b = 2, 4
    x = (np.arange(16)[:, None, None] * 3.0 + r.random((16, 1, c))).astype(np.float16)     # 16 distinct, separated points
    for _ in range(5):
        _, ch = oracle.kmeanspp_init(x, None, r.random((1, 1, 16)), c, b)
        assert sorted(ch[0, 0].tolist()) == list(range(16))


def test_centroid_learning_batches_are_independent_problems():
    # the batched call over heads and groups equals separate calls on each (head, group) slice
    r = np.random.default_rng(10)
    c, b, n, H_, G = 2, 2, 50, 3, 2
    x = r.standard_normal((n, H_, G * c)).astype(np.float16)
    w = r.random((n, H_, G)).astype(np.float32)
    u = r.random((H_, G, 4))
    cb, ch = oracle.kmeanspp_init(x, w, u, c, b)
    new, codes, obj = oracle.lloyd_step(x, w, cb, c, b)
    for h in range(H_):
        for g in range(G):
            xs = np.ascontiguousarray(x[:, h:h + 1, g * c:(g + 1) * c])
            ws = np.ascontiguousarray(w[:, h:h + 1, g:g + 1])
            cb1, ch1 = oracle.kmeanspp_init(xs, ws, u[h:h + 1, g:g + 1], c, b)
            assert ch1[0, 0].tolist() == ch[h, g].tolist()
            n1, c1, o1 = oracle.lloyd_step(xs, ws, cb1, c, b)
            np.testing.assert_array_equal(n1[0, 0], new[h, g])
            np.testing.assert_array_equal(c1[:, 0, 0], codes[:, h, g])
            assert o1[0, 0] == obj[h, g]
