"""Parity at the full workload sizes, in the launch configuration bench.py times.

The caches are built exactly as the benchmark builds them (CUDA encode of seeded synthetic
activations, `bench.DecodeState`).  The oracle cannot recompute a whole workload, so a seeded
sample of (sequence, KV head) items is checked one by one:

* codes: the item's activations are drawn again with the same seeded generator, the oracle
  encodes them on the CPU, and the CUDA codes of the item must match under the near-tie rule;
* attention: the item's slice of the code buffers is overwritten with the ORACLE's codes (so no
  oracle input comes from the CUDA path), the full-size attention call runs, and the item's
  query heads must match the oracle's dense attention within the tolerance.

Items are independent, so the other items of the batch (still CUDA-encoded) cannot influence
the checked outputs.
"""
import numpy as np
import pytest
import torch

import bench
import oracle
import paper_2405_03917_b200 as cq
from paper_2405_03917_b200 import synth
from tests import harness as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def item_activations(w, layer, is_v, head, s, cap):
    """fp16 activations (cap, 128) of sequence s, head `head`, drawn as DecodeState draws them."""
    src = synth.head_source(w.config, layer, head, is_v)
    x = src.activations(w.n_seq * cap, DEV).view(w.n_seq, cap, w.head_dim)[s]
    return x.cpu()


def item_slice(w, cap, s, h):
    nb = (cap + 15) // 16
    size = nb * w.G * (16 + 2 * max(0, w.b - 8))          # bytes of one (sequence, head) in the library layout
    start = (s * w.n_kv_heads + h) * size
    return slice(start, start + size)


def check_items(w, layer, st, items):
    """items: list of (sequence, KV head).  Returns (near_ties, codes_checked, worst max-abs, worst rel-L2)."""
    cap, D, c, b = st.cap, w.head_dim, w.c, w.b
    R = w.n_q_heads // w.n_kv_heads
    ties = total = 0
    oracle_codes = {}
    for (s, h) in items:
        n = int(st.lens_cpu[s])
        assert n >= 1
        for is_v, buf, cb in ((False, st.k_codes, st.k_cb), (True, st.v_codes, st.v_cb)):
            x = item_activations(w, layer, is_v, h, s, cap)                      # (cap, 128) fp16
            cbh = cb[h:h + 1].cpu().numpy()
            res = oracle.encode(x.numpy().reshape(cap, 1, D), cbh, c, b)
            got = cq.cq_codes_to_rowmajor(buf[item_slice(w, cap, s, h)].clone(), 1, cap, 1, D, c, b).cpu().numpy()
            if b > 8:
                got = got.view(np.uint16)
            t, tot = H.check_codes(x.numpy().reshape(cap, 1, D), cbh, got.reshape(cap, 1, w.G), c, b, res)
            ties += t
            total += tot
            oracle_codes[(s, h, is_v)] = res[0].reshape(1, cap, 1, w.G)
            # the attention below reads the oracle's codes for this item
            rm = res[0].astype(np.uint8) if b <= 8 else res[0].astype(np.uint16).view(np.int16)
            patched = cq.cq_codes_from_rowmajor(torch.from_numpy(rm.reshape(1, cap, 1, w.G)).to(DEV), D, c, b)
            buf[item_slice(w, cap, s, h)] = patched
    out = cq.cq_decode_attn(st.q, st.k_codes, st.v_codes, st.k_cb, st.v_cb, st.seq_lens, st.scale, c, b, cap,
                            out=st.out, workspace=st.ws)
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    worst_abs = worst_rel = 0.0
    for (s, h) in items:
        n = int(st.lens_cpu[s])
        q = st.q[s, h * R:(h + 1) * R].cpu().numpy().reshape(1, R, D)
        ref = oracle.decode_dense(q, oracle_codes[(s, h, False)], oracle_codes[(s, h, True)],
                                  st.k_cb[h:h + 1].cpu().numpy(), st.v_cb[h:h + 1].cpu().numpy(),
                                  np.array([n], np.int32), st.scale, c, b)
        a, r = H.check_attn(out[s, h * R:(h + 1) * R], ref[0], f"{w.name} item (seq {s}, kv head {h})")
        worst_abs, worst_rel = max(worst_abs, a), max(worst_rel, r)
    return ties, total, worst_abs, worst_rel


def seeded_items(w, n_items, seed, must=()):
    rng = np.random.default_rng(seed)
    items = list(must)
    while len(items) < n_items:
        it = (int(rng.integers(w.n_seq)), int(rng.integers(w.n_kv_heads)))
        if it not in items:
            items.append(it)
    return items


def test_config1_llama2_7b_4c8b_decode_full_size():
    w = synth.WORKLOADS[1]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    ties, total, a, r = check_items(w, 0, st, seeded_items(w, 64, 101))       # 64 items = 64 query heads x 4096 tokens
    assert ties <= total // 500
    print(f"config 1: {total} codes checked, {ties} near-ties, attention max-abs {a:.2e} rel-L2 {r:.2e}")


def test_config2_mistral_gqa_8c8b_decode_full_size():
    w = synth.WORKLOADS[2]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    # 6 KV heads = 24 query heads x 16384 tokens; one of them among the last items, whose context the
    # launch plan spreads over two CTAs
    ties, total, a, r = check_items(w, 0, st, seeded_items(w, 6, 202, must=[(w.n_seq - 1, 3)]))
    assert ties <= total // 500
    print(f"config 2: {total} codes checked, {ties} near-ties, attention max-abs {a:.2e} rel-L2 {r:.2e}")


def test_config3_2c8b_prefill_encode_full_size():
    w = synth.WORKLOADS[3]
    D, c, b = w.head_dim, w.c, w.b
    rng = np.random.default_rng(303)
    for is_v in (False, True):
        x = synth.layer_activations(w, 0, is_v, w.n_seq, w.n_tokens, device=DEV)
        cb = synth.layer_codebooks(w, 0, is_v).to(DEV)
        buf = torch.zeros(cq.cq_codes_bytes(w.n_seq, w.n_tokens, w.n_kv_heads, D, c, b), dtype=torch.uint8, device=DEV)
        cq.cq_encode(x, cb, c, b, buf, w.n_tokens)
        torch.cuda.synchronize()
        ties = total = 0
        for _ in range(8):                                                    # 8 x 8192 = 65536 vectors per tensor
            s, h = int(rng.integers(w.n_seq)), int(rng.integers(w.n_kv_heads))
            xs = x[s, :, h].cpu().numpy().reshape(w.n_tokens, 1, D)
            got = cq.cq_codes_to_rowmajor(buf[item_slice(w, w.n_tokens, s, h)].clone(), 1, w.n_tokens, 1, D, c, b)
            t, tot = H.check_codes(xs, cb[h:h + 1].cpu().numpy(), got.cpu().numpy().reshape(w.n_tokens, 1, w.G), c, b)
            ties += t
            total += tot
        assert ties <= total // 500
        print(f"config 3 {'V' if is_v else 'K'}: {total} codes checked, {ties} near-ties")
        del x, buf


def test_config4_llama2_13b_8c8b_layers_full_size():
    # 8 of the 40 layers, each at the full per-layer shape (32 sequences x 40 heads, seeded lengths in
    # [8192, 32768]); two items per layer, the shortest or the longest sequence among them
    w = synth.WORKLOADS[4]
    lens = w.lengths()
    s_short, s_long = int(lens.argmin()), int(lens.argmax())
    worst = (0.0, 0.0)
    for k, layer in enumerate((0, 5, 11, 17, 23, 29, 34, 39)):
        st = bench.DecodeState(w, layer, torch.device(DEV), cq)
        rng = np.random.default_rng(400 + layer)
        must = [((s_short if k % 2 == 0 else s_long), int(rng.integers(w.n_kv_heads)))]
        ties, total, a, r = check_items(w, layer, st, seeded_items(w, 2, 404 + layer, must))
        assert ties <= total // 500
        worst = (max(worst[0], a), max(worst[1], r))
        del st
        torch.cuda.empty_cache()
    print(f"config 4: worst attention max-abs {worst[0]:.2e} rel-L2 {worst[1]:.2e}")


def test_config5_llama2_7b_8c10b_decode_full_size():
    # CQ-8c10b (not one of the measured configurations of the headline metric): the wide-code encode and the
    # tuned 1024-centroid attention at the size the benchmark times them, four sampled (sequence, head) items
    w = synth.WORKLOADS[5]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    ties, total, a, r = check_items(w, 0, st, seeded_items(w, 4, 505))
    assert ties <= total // 500
    print(f"config 5: {total} codes checked, {ties} near-ties, attention max-abs {a:.2e} rel-L2 {r:.2e}")


def test_config6_llama2_7b_2c8b_decode_full_size():
    # CQ-2c8b decode (64 groups) at the size the benchmark times it: eight sampled (sequence, head) items
    w = synth.WORKLOADS[6]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    ties, total, a, r = check_items(w, 0, st, seeded_items(w, 8, 606))
    assert ties <= total // 500
    print(f"config 6: {total} codes checked, {ties} near-ties, attention max-abs {a:.2e} rel-L2 {r:.2e}")


def test_prefill_chunk_full_size():
    # cq_prefill_attn at the size the benchmark times it (4 sequences x 8192 cached tokens, the newest 2048 as
    # queries, 32 query heads on 8 KV heads, CQ-8c8b).  Row i of a sequence is Eq. 1 for one query over the first
    # len - n_q + i + 1 tokens: sampled rows of sampled (sequence, KV head) items are checked against the oracle's
    # single-query attention over that prefix, with the oracle's own codes in the items' cache slices.
    w0 = synth.WORKLOADS[2]
    n_seq, cap, n_q = 4, 8192, 2048
    w = synth.Workload("prefill_mistral_7b_gqa_8c8b_chunk2048_of_8192", 8, w0.c, w0.b, 1, n_seq, w0.n_q_heads, w0.n_kv_heads, cap)
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    D, c, b, R = w.head_dim, w.c, w.b, w.n_q_heads // w.n_kv_heads
    items = seeded_items(w, 3, 808)
    oracle_codes = {}
    for (s, h) in items:
        for is_v, buf, cb in ((False, st.k_codes, st.k_cb), (True, st.v_codes, st.v_cb)):
            x = item_activations(w, 0, is_v, h, s, cap)
            res = oracle.encode(x.numpy().reshape(cap, 1, D), cb[h:h + 1].cpu().numpy(), c, b)
            oracle_codes[(s, h, is_v)] = res[0].reshape(1, cap, 1, w.G)
            patched = cq.cq_codes_from_rowmajor(torch.from_numpy(res[0].astype(np.uint8).reshape(1, cap, 1, w.G)).to(DEV), D, c, b)
            buf[item_slice(w, cap, s, h)] = patched
    g = torch.Generator(device="cpu").manual_seed(88)
    q = torch.randn(n_seq, n_q, w.n_q_heads, D, generator=g).to(torch.float16)
    out = cq.cq_prefill_attn(q.to(DEV), st.k_codes, st.v_codes, st.k_cb, st.v_cb, st.seq_lens, st.scale, c, b, cap)
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    rng = np.random.default_rng(809)
    worst_abs = worst_rel = 0.0
    for (s, h) in items:
        n = int(st.lens_cpu[s])
        # first and last query, the rows around a 64-token tile edge and a 32-query row-tile edge, and random ones
        rows = sorted({0, 1, 31, 32, 63, 64, n_q - 1} | {int(v) for v in rng.integers(0, n_q, size=9)})
        for i in rows:
            prefix = n - n_q + i + 1
            if prefix < 1:
                assert (out[s, i, h * R:(h + 1) * R] == 0).all()
                continue
            qr = q[s, i, h * R:(h + 1) * R].numpy().reshape(1, R, D)
            ref = oracle.decode_dense(qr, oracle_codes[(s, h, False)], oracle_codes[(s, h, True)],
                                      st.k_cb[h:h + 1].cpu().numpy(), st.v_cb[h:h + 1].cpu().numpy(),
                                      np.array([prefix], np.int32), st.scale, c, b)
            a, r = H.check_attn(out[s, i, h * R:(h + 1) * R], ref[0], f"prefill item (seq {s}, kv head {h}) row {i}")
            worst_abs, worst_rel = max(worst_abs, a), max(worst_rel, r)
    print(f"prefill: {len(items)} items, attention max-abs {worst_abs:.2e} rel-L2 {worst_rel:.2e}")


def test_pre_rope_decode_full_size():
    # cq_decode_attn_rope on config 1's shape (16 x 32 heads x 4096 tokens, CQ-4c8b, the tuned kernel), with the
    # rotary tables of base 10000 that the benchmark uses: sampled (sequence, head) items against the oracle's
    # dequantise-rotate-attend form, the oracle's own codes in the items' cache slices.
    w = synth.WORKLOADS[1]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    cap, D, c, b = st.cap, w.head_dim, w.c, w.b
    R = w.n_q_heads // w.n_kv_heads
    items = seeded_items(w, 12, 909)
    oracle_codes = {}
    for (s, h) in items:
        for is_v, buf, cb in ((False, st.k_codes, st.k_cb), (True, st.v_codes, st.v_cb)):
            x = item_activations(w, 0, is_v, h, s, cap)
            res = oracle.encode(x.numpy().reshape(cap, 1, D), cb[h:h + 1].cpu().numpy(), c, b)
            oracle_codes[(s, h, is_v)] = res[0].reshape(1, cap, 1, w.G)
            patched = cq.cq_codes_from_rowmajor(torch.from_numpy(res[0].astype(np.uint8).reshape(1, cap, 1, w.G)).to(DEV), D, c, b)
            buf[item_slice(w, cap, s, h)] = patched
    P = D // 2
    ang = np.arange(cap, dtype=np.float64)[:, None] * (10000.0 ** (-np.arange(P, dtype=np.float64) / P))[None, :]
    cs, sn = np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
    out = cq.cq_decode_attn_rope(st.q, st.k_codes, st.v_codes, st.k_cb, st.v_cb, st.seq_lens, torch.from_numpy(cs).to(DEV),
                                 torch.from_numpy(sn).to(DEV), st.scale, c, b, cap, workspace=st.ws, variant=2)
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    worst_abs = worst_rel = 0.0
    for (s, h) in items:
        n = int(st.lens_cpu[s])
        q = st.q[s, h * R:(h + 1) * R].cpu().numpy().reshape(1, R, D)
        ref = oracle.decode_dense_rope(q, oracle_codes[(s, h, False)], oracle_codes[(s, h, True)],
                                       st.k_cb[h:h + 1].cpu().numpy(), st.v_cb[h:h + 1].cpu().numpy(),
                                       np.array([n], np.int32), cs, sn, st.scale, c, b)
        a, r = H.check_attn(out[s, h * R:(h + 1) * R], ref[0], f"pre-RoPE item (seq {s}, head {h})")
        worst_abs, worst_rel = max(worst_abs, a), max(worst_rel, r)
    print(f"pre-RoPE decode: {len(items)} items, attention max-abs {worst_abs:.2e} rel-L2 {worst_rel:.2e}")


@pytest.mark.parametrize("wi,n_items,seed", [(2, 4, 212), (4, 4, 414), (1, 8, 111)])
def test_decode_step_full_size(wi, n_items, seed):
    # The call the benchmark times: cq_decode_step (the new token's K and V are encoded and written at the last
    # position inside the attention launch, which then attends over all tokens), on config 2 (the kernel with two
    # heads per table word, one launch), on config 4's ragged layer and on config 1 (the appending instances of the
    # one-head-per-word kernel).  Sampled (sequence, KV head) items hold the oracle's codes; afterwards the
    # appended codes must be the oracle's codes of the new vectors (near-tie rule) and the outputs the oracle's
    # attention over the updated cache.
    w = synth.WORKLOADS[wi]
    st = bench.DecodeState(w, 0, torch.device(DEV), cq)
    assert st.fused_launches <= 2 and (wi != 2 or st.fused_launches == 1)
    cap, D, c, b = st.cap, w.head_dim, w.c, w.b
    R = w.n_q_heads // w.n_kv_heads
    items = seeded_items(w, n_items, seed, must=[(w.n_seq - 1, w.n_kv_heads - 3)])
    codes = {}
    for (s, h) in items:
        for is_v, buf, cb in ((False, st.k_codes, st.k_cb), (True, st.v_codes, st.v_cb)):
            x = item_activations(w, 0, is_v, h, s, cap)
            res = oracle.encode(x.numpy().reshape(cap, 1, D), cb[h:h + 1].cpu().numpy(), c, b)
            codes[(s, h, is_v)] = res[0].reshape(1, cap, 1, w.G).copy()
            buf[item_slice(w, cap, s, h)] = cq.cq_codes_from_rowmajor(
                torch.from_numpy(res[0].astype(np.uint8).reshape(1, cap, 1, w.G)).to(DEV), D, c, b)
    st.step(cq)
    torch.cuda.synchronize()
    out = st.out.cpu().numpy()
    ties = total = 0
    worst_abs = worst_rel = 0.0
    for (s, h) in items:
        n = int(st.lens_cpu[s])
        for is_v, buf, cb, new in ((False, st.k_codes, st.k_cb, st.k_new), (True, st.v_codes, st.v_cb, st.v_new)):
            xn = new[s, h].cpu().numpy().reshape(1, 1, D)
            cbh = cb[h:h + 1].cpu().numpy()
            res = oracle.encode(xn, cbh, c, b)
            got = cq.cq_codes_to_rowmajor(buf[item_slice(w, cap, s, h)].clone(), 1, cap, 1, D, c, b).cpu().numpy()
            got = got.reshape(cap, w.G)
            t, tot = H.check_codes(xn, cbh, got[n - 1].reshape(1, 1, w.G), c, b, res)
            ties += t
            total += tot
            # every other position of the item is untouched
            keep = codes[(s, h, is_v)].reshape(cap, w.G)
            assert (got[:n - 1] == keep[:n - 1]).all() and (got[n:] == keep[n:]).all()
            codes[(s, h, is_v)][0, n - 1, 0] = res[0].reshape(w.G)
        q = st.q[s, h * R:(h + 1) * R].cpu().numpy().reshape(1, R, D)
        ref = oracle.decode_dense(q, codes[(s, h, False)], codes[(s, h, True)], st.k_cb[h:h + 1].cpu().numpy(),
                                  st.v_cb[h:h + 1].cpu().numpy(), np.array([n], np.int32), st.scale, c, b)
        a, r = H.check_attn(out[s, h * R:(h + 1) * R], ref[0], f"step item (seq {s}, kv head {h})")
        worst_abs, worst_rel = max(worst_abs, a), max(worst_rel, r)
    assert ties <= 1
    print(f"config {wi} step: {total} appended codes checked, {ties} near-ties, attention max-abs {worst_abs:.2e} rel-L2 {worst_rel:.2e}")
