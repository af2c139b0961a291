"""GPU parity of cq_decode_step (the new token encoded and appended inside the attention launch where the
shape has such a kernel, as two launches elsewhere) against the fp64 CPU oracle and against the separate
cq_encode_kv + cq_decode_attn calls."""
import numpy as np
import pytest
import torch

import oracle
import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_case(seed, c, b, n_seq, n_q, n_kv, cap):
    w = H.small_workload("step", seed, c, b, n_seq, n_q, n_kv, cap)
    xk = synth.layer_activations(w, 0, False, n_seq, cap)
    xv = synth.layer_activations(w, 0, True, n_seq, cap)
    kcb, vcb = synth.layer_codebooks(w, 0, False), synth.layer_codebooks(w, 0, True)
    q = synth.queries(seed, 0, n_seq, n_q)
    return xk, xv, kcb, vcb, q


def encode_cache(x, cb, c, b, cap):
    n_seq, _, n_heads, D = x.shape
    buf = torch.zeros(cq.cq_codes_bytes(n_seq, cap, n_heads, D, c, b), dtype=torch.uint8, device=DEV)
    cq.cq_encode(x.to(DEV), cb.to(DEV), c, b, buf, cap)
    return buf


def step_and_check(c, b, n_q, n_kv, cap, lens, seed, what):
    """One step on caches that hold the tokens of xk / xv; the new token of sequence s is row (7, 9) of it."""
    n_seq, D = len(lens), 128
    xk, xv, kcb, vcb, q = make_case(seed, c, b, n_seq, n_q, n_kv, cap)
    kbuf, vbuf = encode_cache(xk, kcb, c, b, cap), encode_cache(xv, vcb, c, b, cap)
    k_new = torch.stack([xk[s, 7 % cap] for s in range(n_seq)]).contiguous()
    v_new = torch.stack([xv[s, 9 % cap] for s in range(n_seq)]).contiguous()
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kd, vd = kcb.to(DEV), vcb.to(DEV)

    # the same step as two calls on copies of the caches
    kref, vref = kbuf.clone(), vbuf.clone()
    cq.cq_encode_kv(k_new[:, None].contiguous().to(DEV), v_new[:, None].contiguous().to(DEV), kd, vd, c, b, kref, vref, cap,
                    seq_offsets=sl)
    sl1 = torch.tensor([min(n + 1, cap) for n in lens], dtype=torch.int32, device=DEV)
    want = cq.cq_decode_attn(q.to(DEV), kref, vref, kd, vd, sl1, D ** -0.5, c, b, cap).cpu().numpy()

    got = cq.cq_decode_step(q.to(DEV), k_new.to(DEV), v_new.to(DEV), sl, kbuf, vbuf, kd, vd, D ** -0.5, c, b, cap).cpu().numpy()
    assert torch.equal(kbuf, kref) and torch.equal(vbuf, vref), f"{what}: caches differ from cq_encode_kv's"
    assert torch.equal(sl.cpu(), torch.tensor(lens, dtype=torch.int32)), "seq_lens must not be modified"

    # oracle: the new token written at position lens[s], context lens[s] + 1 (a full sequence gets no new token)
    xk2, xv2 = xk.clone(), xv.clone()
    for s, n in enumerate(lens):
        if n < cap:
            xk2[s, n], xv2[s, n] = k_new[s], v_new[s]
    kc_rm, _ = H.oracle_encode_rowmajor(xk2, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv2, vcb, c, b)
    ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), sl1.cpu().numpy(), D ** -0.5, c, b)
    for s in range(n_seq):
        H.check_attn(got[s], ref[s], f"{what} seq {s} (len {lens[s]}) vs oracle")
        H.check_attn(got[s], want[s], f"{what} seq {s} (len {lens[s]}) vs two calls")
    got_k = cq.cq_codes_to_rowmajor(kbuf, n_seq, cap, n_kv, D, c, b).cpu().numpy()
    got_v = cq.cq_codes_to_rowmajor(vbuf, n_seq, cap, n_kv, D, c, b).cpu().numpy()
    for s, n in enumerate(lens):
        if n < cap:
            H.check_codes(k_new[s:s + 1].numpy(), kcb.numpy(), got_k[s, n][None], c, b)
            H.check_codes(v_new[s:s + 1].numpy(), vcb.numpy(), got_v[s, n][None], c, b)


@pytest.mark.parametrize("n_q,n_kv", [(8, 2), (4, 1), (16, 2)])
def test_append_inside_the_attention_launch(n_q, n_kv):
    # CQ-8c8b with four (or eight) query heads per KV head: the kernel that appends inside the launch.
    # Lengths: empty cache, last slot of a block, first slot of a block, inside the first tile, inside a later
    # tile of another warp, one short of capacity, at capacity (no new token).
    cap = 1100
    lens = [0, 15, 16, 37, 64 * 9 + 5, 1000, cap - 1, cap]
    step_and_check(8, 8, n_q, n_kv, cap, lens, 5 + n_q, f"fused Hq={n_q} Hkv={n_kv}")


def test_append_with_a_context_split_over_several_ctas():
    # few sequences with long contexts: the plan spreads each over several CTAs; the new token lies in the last
    # part, at its start, or alone in a part of its own
    cap = 20000
    plan_chunk = 512
    lens = [19999, 12 * plan_chunk, 12 * plan_chunk - 1, 7001]
    step_and_check(8, 8, 8, 2, cap, lens, 77, "split context")


@pytest.mark.parametrize("c,b,n_q,n_kv", [(4, 8, 4, 4), (8, 8, 2, 2), (2, 8, 4, 2), (8, 10, 2, 1), (8, 8, 6, 2)])
def test_step_on_shapes_without_the_fused_kernel(c, b, n_q, n_kv):
    cap = 300
    step_and_check(c, b, n_q, n_kv, cap, [0, 31, 299, 300, 128], 11 * c + b, f"two launches c={c} b={b}")


def test_steps_in_a_row_build_the_cache_the_oracle_encodes():
    # 40 steps from an empty cache: afterwards the cache holds the oracle's codes of the 40 tokens and every
    # step's output was the attention over the tokens so far
    c, b, D, cap, n_seq, n_q, n_kv, steps = 8, 8, 128, 64, 2, 8, 2, 40
    xk, xv, kcb, vcb, _ = make_case(3, c, b, n_seq, n_q, n_kv, cap)
    kd, vd = kcb.to(DEV), vcb.to(DEV)
    nbytes = cq.cq_codes_bytes(n_seq, cap, n_kv, D, c, b)
    kbuf, vbuf = (torch.zeros(nbytes, dtype=torch.uint8, device=DEV) for _ in range(2))
    kc_rm, _ = H.oracle_encode_rowmajor(xk, kcb, c, b)
    vc_rm, _ = H.oracle_encode_rowmajor(xv, vcb, c, b)
    g = torch.Generator().manual_seed(9)
    for t in range(steps):
        q = torch.randn(n_seq, n_q, D, generator=g).to(torch.float16)
        sl = torch.full((n_seq,), t, dtype=torch.int32, device=DEV)
        out = cq.cq_decode_step(q.to(DEV), xk[:, t].contiguous().to(DEV), xv[:, t].contiguous().to(DEV), sl, kbuf, vbuf,
                                kd, vd, D ** -0.5, c, b, cap).cpu().numpy()
        if t in (0, 1, 15, 16, 39):
            ref = oracle.decode_dense(q.numpy(), kc_rm, vc_rm, kcb.numpy(), vcb.numpy(), np.full(n_seq, t + 1, np.int32),
                                      D ** -0.5, c, b)
            H.check_attn(out, ref, f"step {t}")
    got_k = cq.cq_codes_to_rowmajor(kbuf, n_seq, cap, n_kv, D, c, b).cpu().numpy()[:, :steps]
    got_v = cq.cq_codes_to_rowmajor(vbuf, n_seq, cap, n_kv, D, c, b).cpu().numpy()[:, :steps]
    H.check_codes(xk[:, :steps].numpy().reshape(-1, n_kv, D), kcb.numpy(), got_k.reshape(-1, n_kv, D // c), c, b)
    H.check_codes(xv[:, :steps].numpy().reshape(-1, n_kv, D), vcb.numpy(), got_v.reshape(-1, n_kv, D // c), c, b)


def test_bad_arguments_are_refused():
    c, b, D, cap, n_seq, n_q, n_kv = 8, 8, 128, 50, 2, 8, 2
    xk, xv, kcb, vcb, q = make_case(1, c, b, n_seq, n_q, n_kv, cap)
    kbuf, vbuf = encode_cache(xk, kcb, c, b, cap), encode_cache(xv, vcb, c, b, cap)
    sl = torch.tensor([3, 4], dtype=torch.int32, device=DEV)
    k_new, v_new = xk[:, 0].contiguous().to(DEV), xv[:, 0].contiguous().to(DEV)
    with pytest.raises(ValueError):                      # key of the wrong shape
        cq.cq_decode_step(q.to(DEV), k_new[:, :1], v_new, sl, kbuf, vbuf, kcb.to(DEV), vcb.to(DEV), 0.1, c, b, cap)
    with pytest.raises(ValueError):                      # undersized cache
        cq.cq_decode_step(q.to(DEV), k_new, v_new, sl, kbuf[:64], vbuf, kcb.to(DEV), vcb.to(DEV), 0.1, c, b, cap)
    with pytest.raises(cq.CQError):                      # workspace too small
        cq.cq_decode_step(q.to(DEV), k_new, v_new, sl, kbuf, vbuf, kcb.to(DEV), vcb.to(DEV), 0.1, c, b, cap,
                          workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    with pytest.raises(cq.CQError):                      # the two caches must be different buffers
        cq.cq_decode_step(q.to(DEV), k_new, v_new, sl, kbuf, kbuf, kcb.to(DEV), vcb.to(DEV), 0.1, c, b, cap)
