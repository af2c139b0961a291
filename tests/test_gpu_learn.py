"""GPU parity of centroid learning (Section 3.2.1) against the fp64 CPU oracle.

* k-means++: the chosen centres are integers decided from fp64 sums that both sides form in the
  same order, so the initial codebooks must be equal bit for bit;
* one k-means iteration from a common state: the assignment is cq_encode (near-tie rule), the
  new centroids and the objective match within fp32-accumulation tolerance;
* a whole run: k-means trajectories are chaotic in the last bits, so the unique things are
  compared: the objective never increases, and ends within a percent of the oracle's run from the
  same initial centroids.
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


def calib(config, n_vec, n_heads, is_v, c):
    w = H.small_workload("learn", config, c, 8, 1, n_heads, n_heads, n_vec)
    x = synth.layer_activations(w, 0, is_v, 1, n_vec)[0].contiguous()          # (n_vec, n_heads, 128) fp16
    return x


def fisher_like_weights(seed, n_vec, n_heads, G):
    # stand-in for the per-group squared gradient norms of Eq. 6: positive, heavy-tailed
    g = torch.Generator().manual_seed(seed)
    return torch.randn(n_vec, n_heads, G, generator=g).pow(2).mul(torch.rand(n_vec, 1, 1, generator=g) * 3 + 0.1).float()


@pytest.mark.parametrize("c,b,n_heads,n_vec,weighted", [(8, 8, 2, 1500, False), (4, 8, 1, 700, True), (2, 8, 2, 900, True),
                                                       (8, 5, 3, 300, False), (4, 2, 2, 64, True)])
def test_kmeanspp_init_is_bit_equal(c, b, n_heads, n_vec, weighted):
    x = calib(300 + c, n_vec, n_heads, False, c)
    G = 128 // c
    w = fisher_like_weights(c * b, n_vec, n_heads, G) if weighted else None
    if weighted:
        w[::7] = 0                                                       # vectors that must never be drawn
    u = torch.rand(n_heads, G, 1 << b, dtype=torch.float64, generator=torch.Generator().manual_seed(b))
    want, chosen = oracle.kmeanspp_init(x.numpy(), None if w is None else w.numpy(), u.numpy(), c, b)
    got = cq.cq_kmeanspp_init(x.to(DEV), None if w is None else w.to(DEV), u.to(DEV), c, b).cpu().numpy()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("c,b,n_vec,weighted", [(8, 8, 5000, True), (4, 6, 4096, False), (8, 4, 6200, True), (2, 5, 2049, False)])
def test_kmeanspp_init_is_bit_equal_over_several_tiles(c, b, n_vec, weighted):
    # more vectors than one tile of the draw's in-order sum (2048): the running sums kept at the tile ends decide
    # where the walk for the drawn vector starts; uniforms at both ends of [0, 1) and runs of zero contributions
    # (whole tiles of them in the weighted cases) are part of the input
    x = calib(340 + c, n_vec, 1, False, c)
    G = 128 // c
    w = fisher_like_weights(c + b, n_vec, 1, G) if weighted else None
    if weighted:
        w[::5] = 0
        w[:2100] = 0                                                     # the first tile, and part of the second
        w[4200:4900] = 0
    u = torch.rand(1, G, 1 << b, dtype=torch.float64, generator=torch.Generator().manual_seed(40 + b))
    u[0, :, 1] = 0.0
    u[0, :, 2] = 1.0 - 2.0 ** -53
    u[0, ::2, 3] = 2.0 ** -40
    want, chosen = oracle.kmeanspp_init(x.numpy(), None if w is None else w.numpy(), u.numpy(), c, b)
    got = cq.cq_kmeanspp_init(x.to(DEV), None if w is None else w.to(DEV), u.to(DEV), c, b).cpu().numpy()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("c,b,n_heads,n_vec,weighted", [(8, 8, 2, 3000, False), (8, 8, 2, 3000, True), (4, 8, 2, 2000, True),
                                                       (2, 8, 1, 2500, False), (8, 4, 2, 500, True)])
def test_one_iteration_from_common_state(c, b, n_heads, n_vec, weighted):
    x = calib(310 + c, n_vec, n_heads, True, c)
    G = 128 // c
    w = fisher_like_weights(7 * c + b, n_vec, n_heads, G) if weighted else None
    u = np.random.default_rng(c + b).random((n_heads, G, 1 << b))
    cb0, _ = oracle.kmeanspp_init(x.numpy(), None if w is None else w.numpy(), u, c, b)
    want, codes, obj = oracle.lloyd_step(x.numpy(), None if w is None else w.numpy(), cb0, c, b)
    got, gobj = cq.cq_lloyd_step(x.to(DEV), None if w is None else w.to(DEV), torch.from_numpy(cb0).to(DEV), c, b)
    got, gobj = got.cpu().numpy(), gobj.cpu().numpy()
    # The assignment is cq_encode: inside the near-tie band it may give a vector to another centroid than
    # the oracle does.  Those vectors are named (the GPU's own assignment against the oracle's) and the
    # centroids that gain or lose one of them are set aside; every other centroid has the same members on
    # both sides and must agree within fp32 accumulation of up to n_vec terms.
    buf = torch.zeros(cq.cq_codes_bytes(1, n_vec, n_heads, 128, c, b), dtype=torch.uint8, device=DEV)
    cq.cq_encode(x.view(1, n_vec, n_heads, 128).to(DEV), torch.from_numpy(cb0).to(DEV), c, b, buf, n_vec)
    gcodes = cq.cq_codes_to_rowmajor(buf, 1, n_vec, n_heads, 128, c, b).cpu().numpy().astype(np.int64)[0]
    moved = gcodes != codes                                              # (n_vec, n_heads, G)
    H.check_codes(x.numpy(), cb0, gcodes, c, b)                          # ... and every move is a near-tie
    touched = np.zeros(want.shape[:3], dtype=bool)                       # (n_heads, G, 2^b)
    v, h, g = np.nonzero(moved)
    touched[h, g, gcodes[v, h, g]] = True
    touched[h, g, codes[v, h, g]] = True
    assert moved.sum() <= max(2, moved.size // 2000), f"{moved.sum()} of {moved.size} vectors moved"
    scale = np.abs(want).max()
    close = np.abs(got - want) <= 2e-5 * scale + 2e-5 * np.abs(want)
    bad = ~close & ~touched[..., None]
    assert not bad.any(), f"{bad.sum()} centroid components differ although their members are the same"
    np.testing.assert_allclose(gobj, obj, rtol=1e-5)


def test_learning_run_descends_and_matches_the_oracle_objective():
    c, b, n_heads, n_vec, iters = 8, 6, 2, 4000, 12
    x = calib(333, n_vec, n_heads, False, c)
    G = 128 // c
    w = fisher_like_weights(5, n_vec, n_heads, G)
    u = np.random.default_rng(3).random((n_heads, G, 1 << b))
    xd, wd = x.to(DEV), w.to(DEV)
    cb = cq.cq_kmeanspp_init(xd, wd, torch.from_numpy(u).to(DEV), c, b)
    ocb, _ = oracle.kmeanspp_init(x.numpy(), w.numpy(), u, c, b)
    assert np.array_equal(cb.cpu().numpy(), ocb)
    last = None
    for _ in range(iters):
        cb, obj = cq.cq_lloyd_step(xd, wd, cb, c, b)
        o = obj.cpu().numpy()
        if last is not None:
            assert (o <= last * (1 + 1e-6)).all()
        last = o
        ocb, _, oobj = oracle.lloyd_step(x.numpy(), w.numpy(), ocb, c, b)
    np.testing.assert_allclose(last, oobj, rtol=1e-2)
    # the one-call driver gives the same objective as the step-by-step run
    cb2, obj2 = cq.cq_learn_centroids(xd, wd, torch.from_numpy(u).to(DEV), c, b, iters)
    np.testing.assert_allclose(obj2.cpu().numpy(), last, rtol=1e-2)
    # and the learned codebooks do what they are for: a lower quantisation error than the initial ones
    codes, d_best, _ = oracle.encode(x.numpy(), cb2.cpu().numpy(), c, b)
    _, d_init, _ = oracle.encode(x.numpy(), oracle.kmeanspp_init(x.numpy(), w.numpy(), u, c, b)[0], c, b)
    assert (w.numpy() * d_best).sum() < 0.8 * (w.numpy() * d_init).sum()
