#!/usr/bin/env python
"""Benchmark of the CQ hot path on B200.

One "step" is one decode step over every layer of the workload (default: CQ-8c8b on a
Mistral-7B-shaped GQA layer, batch 64, context 16384, one layer): per layer the new token's
key and value vectors are CQ-encoded and appended and every query head attends over the coded
cache (cq_decode_step: one launch where the attention kernel appends the token itself, else
cq_encode_kv followed by cq_decode_attn).  Inputs are seeded and synthetic.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2|cfg1|cfg4|cfg0] [--extras none|default|decode|all]

Prints ONE JSON line (rank 0).  `value` is KV tokens/s with everything resident in HBM;
`e2e` is the same metric through cq_decode_step_host with host buffers; `roofline` describes
the decode-attention call against the two ceilings it has - the measured HBM copy bandwidth
and the SMs' shared-memory pipe - names the lower one as the bound and carries both
fractions; `cpu_baseline` is the fp64 CPU oracle on a bounded sample.  With --impl reference the oracle itself is the timed arm.
Under torchrun every rank runs its own replica of the batch (weak scaling, no collective
on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_03917_b200 import synth  # noqa: E402

HBM_FALLBACK_GBS = 6650.0
METRIC = "cq_decode_attn_kv_tokens_per_s"
UNIT = "KV tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback"


def kernel_source_hash(files=("cq_decode.cu", "cq_decode_pair.cu", "cq_decode_util.cuh", "cq_bulk_copy.cuh", "cq_common.cuh")):
    """sha256 over the source files of a decode kernel (the kernel a roofline object describes)."""
    import hashlib
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, "paper_2405_03917_b200", "csrc", f), "rb").read())
    return h.hexdigest()


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local)
        dist.init_process_group(backend=backend)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------- setup

class DecodeState:
    """Device-resident coded cache of one layer of a workload, built with the CUDA encode."""

    def __init__(self, w: synth.Workload, layer: int, dev, cq, lens=None):
        self.w, self.dev = w, dev
        D, c, b = w.head_dim, w.c, w.b
        self.lens_cpu = w.lengths() if lens is None else lens
        self.cap = w.n_tokens
        nbytes = cq.cq_codes_bytes(w.n_seq, self.cap, w.n_kv_heads, D, c, b)
        self.k_codes = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        self.v_codes = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
        self.k_cb = synth.layer_codebooks(w, layer, False).to(dev)
        self.v_cb = synth.layer_codebooks(w, layer, True).to(dev)
        # encode head by head so that at most one head's activations are alive
        for is_v, codes, cb in ((False, self.k_codes, self.k_cb), (True, self.v_codes, self.v_cb)):
            x = synth.layer_activations(w, layer, is_v, w.n_seq, self.cap, device=dev)
            cq.cq_encode(x, cb, c, b, codes, self.cap)
            # the step's new token: a fresh draw per (sequence, head)
            new = torch.stack([synth.head_source(w.config, layer, h, is_v).activations(w.n_seq, dev, stream=2)
                               for h in range(w.n_kv_heads)], dim=1).contiguous()
            if is_v:
                self.v_new = new
            else:
                self.k_new = new
            del x
        self.q = synth.queries(w.config, layer, w.n_seq, w.n_q_heads, device=dev)
        self.seq_lens = self.lens_cpu.to(dev)
        self.append_pos = (self.lens_cpu - 1).to(dev)
        self.out = torch.empty(w.n_seq, w.n_q_heads, D, dtype=torch.float32, device=dev)
        self.ws = torch.empty(max(256, cq.cq_decode_step_workspace_bytes(w.n_seq, w.n_q_heads, w.n_kv_heads, D, c, b,
                                                                        self.cap)), dtype=torch.uint8, device=dev)
        self.scale = D ** -0.5
        # launches of one cq_decode_step call: 1 or 2 where the attention kernel appends the token itself
        self.fused_launches = cq.cq_decode_step_launches(w.n_seq, w.n_q_heads, w.n_kv_heads, D, c, b, self.cap)

    def kv_tokens(self) -> int:
        return int(self.lens_cpu.sum().item())

    def algorithmic_bytes(self) -> int:
        """Bytes decode attention must read per call: one byte per (token, KV head, group) for K
        and for V, both codebooks once per KV head, queries; plus the output it writes."""
        w = self.w
        code_bytes_x16 = 16 + 2 * max(0, w.b - 8)               # bytes of 16 codes of one group
        codes = 2 * self.kv_tokens() * w.n_kv_heads * w.G * code_bytes_x16 // 16
        books = 2 * w.n_kv_heads * w.G * (1 << w.b) * w.c * 4
        qo = w.n_seq * w.n_q_heads * w.head_dim * (2 + 4)
        return codes + books + qo

    def attend(self, cq, ev=None):
        """Decode attention alone (cq_decode_attn) over the cache as it stands."""
        w = self.w
        if ev is not None:
            ev[0].record()
        cq.cq_decode_attn(self.q, self.k_codes, self.v_codes, self.k_cb, self.v_cb, self.seq_lens, self.scale,
                          w.c, w.b, self.cap, out=self.out, workspace=self.ws)
        if ev is not None:
            ev[1].record()

    def step(self, cq, ev=None):
        """Append-encode the new token (K, V) at the last position, then attend: one cq_decode_step call where the
        kernel appends inside the attention launch, else cq_encode_kv followed by cq_decode_attn."""
        w = self.w
        if self.fused_launches <= 2:
            if ev is not None:
                ev[0].record()
            cq.cq_decode_step(self.q, self.k_new, self.v_new, self.append_pos, self.k_codes, self.v_codes, self.k_cb,
                              self.v_cb, self.scale, w.c, w.b, self.cap, out=self.out, workspace=self.ws)
            if ev is not None:
                ev[1].record()
            return
        cq.cq_encode_kv(self.k_new.view(w.n_seq, 1, w.n_kv_heads, w.head_dim),
                        self.v_new.view(w.n_seq, 1, w.n_kv_heads, w.head_dim), self.k_cb, self.v_cb, w.c, w.b,
                        self.k_codes, self.v_codes, self.cap, seq_offsets=self.append_pos)
        if ev is not None:
            ev[0].record()
        cq.cq_decode_attn(self.q, self.k_codes, self.v_codes, self.k_cb, self.v_cb, self.seq_lens, self.scale,
                          w.c, w.b, self.cap, out=self.out, workspace=self.ws)
        if ev is not None:
            ev[1].record()


def attach_traffic(roofline, workload_name):
    """DRAM bytes of one launch from the committed ncu counters, when the kernels have not changed since."""
    tr = os.path.join(ROOT, "profiles", "decode_traffic.json")
    if not os.path.exists(tr):
        return
    try:
        t = json.load(open(tr)).get(workload_name)
        # the counters describe one build of the kernels: any later edit of their source voids them
        if t and t.get("kernel_source_sha256") == kernel_source_hash(tuple(t["files"])):
            roofline["traffic"] = t["dram_bytes_per_launch"]
            roofline["traffic_source"] = t.get("source")
    except Exception:
        pass


def shared_word_kernel(w) -> bool:
    """Shapes served by the kernel that keeps two query heads in one table word (cq_decode_pair.cu)."""
    return w.head_dim == 128 and w.b == 8 and w.c == 8 and (w.n_q_heads // w.n_kv_heads) % 4 == 0


def decode_roofline(w, st, ms, dev, sm_mhz=None):
    """The two ceilings of one decode-attention call that took `ms`:
    hbm   - the bytes the call must read (codes addressed by seq_lens, both codebooks once per KV head,
            queries, output) against the measured copy bandwidth;
    smem  - the 4-byte shared-memory lane operations the formulation needs per (token, KV head): one bin
            add per (group, query head) plus the table lookups (one per (group, query head); one per
            (group, two query heads) where a table word holds two heads), against 32 lanes per clock
            and SM at the sampled SM clock.
    `bound` names the ceiling that allows less (the larger minimum time)."""
    hbm, which = measured_peaks()
    props = torch.cuda.get_device_properties(dev)
    n_sm = props.multi_processor_count
    mhz = float(sm_mhz) if sm_mhz else props.clock_rate / 1e3
    R = w.n_q_heads // w.n_kv_heads
    per_tok = w.G * R + (w.G * R // 2 if shared_word_kernel(w) else w.G * R)
    lane_ops = float(per_tok) * st.kv_tokens() * w.n_kv_heads
    smem_peak = n_sm * 32 * mhz * 1e6
    nbytes = st.algorithmic_bytes()
    t_hbm, t_smem = nbytes / (hbm * 1e9), lane_ops / smem_peak
    a_hbm, a_smem = nbytes / (ms * 1e-3) / 1e9, lane_ops / (ms * 1e-3)
    merged = w.b == 10 or st.fused_launches != 1         # a merge launch follows unless the kernel writes the output itself
    o = {"kernel": ("decode_pair_kernel" if shared_word_kernel(w) else
                    "decode_wide_kernel" if w.b == 10 else "decode_tuned_kernel") +
                   (" + merge_kernel (one attention call)" if merged else " (one attention call; the kernel writes the output itself)"),
         "launch_ms": ms, "algorithmic_bytes_per_launch": nbytes, "traffic": None,
         "hbm": {"achieved": a_hbm, "peak": hbm, "unit": "GB/s", "frac": a_hbm / hbm, "frac_of_8tbs_nominal": a_hbm / 8000.0,
                 "peak_source": which + " copy bandwidth", "min_ms": t_hbm * 1e3},
         "smem": {"achieved": a_smem, "peak": smem_peak, "unit": "lane-ops/s", "frac": a_smem / smem_peak,
                  "lane_ops_per_kv_head_token": per_tok, "min_ms": t_smem * 1e3,
                  "peak_source": f"32 lanes/clk/SM x {n_sm} SMs x {mhz:.0f} MHz (sampled SM clock)"}}
    lower = "hbm" if t_hbm >= t_smem else "smem"
    o.update(bound=lower, achieved=o[lower]["achieved"], peak=o[lower]["peak"], unit=o[lower]["unit"], frac=o[lower]["frac"])
    return o


def time_steps(fn, steps, warmup, world, dev):
    for _ in range(warmup):
        fn(None)
    torch.cuda.synchronize()
    barrier(world)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    inner = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    e0.record()
    for i in range(steps):
        fn(inner[i])
    e1.record()
    torch.cuda.synchronize()
    barrier(world)
    total_ms = e0.elapsed_time(e1)
    inner_ms = [a.elapsed_time(b) for a, b in inner]
    return max_over_ranks(total_ms, world, dev), inner_ms


# ----------------------------------------------------------------------------- CPU oracle

def oracle_sample_state(w: synth.Workload, n_sample_seq: int = 1):
    """Oracle-side copy of the first sequences of the workload: the cache is encoded by the
    oracle itself (untimed set-up), never read from the CUDA path."""
    import oracle
    layer = 0
    lens = w.lengths()[:n_sample_seq].numpy().astype(np.int32)
    cap = int(lens.max())
    st = {"lens": lens, "cap": cap}
    # CPU and CUDA generators give different draws of the same distribution, so the sample is
    # drawn directly at its own size.
    for is_v, key in ((False, "k"), (True, "v")):
        cb = synth.layer_codebooks(w, layer, is_v).numpy()
        x = synth.layer_activations(w, layer, is_v, n_sample_seq, cap)
        xn = x.numpy().reshape(n_sample_seq * cap, w.n_kv_heads, w.head_dim)
        codes, _, _ = oracle.encode(xn, cb, w.c, w.b)
        st[key + "_cb"] = cb
        st[key + "_codes"] = codes.reshape(n_sample_seq, cap, w.n_kv_heads, w.G)
        new = torch.stack([synth.head_source(w.config, layer, h, is_v).activations(w.n_seq, "cpu", stream=2)
                           for h in range(w.n_kv_heads)], dim=1)[:n_sample_seq]
        st[key + "_new"] = new.numpy().reshape(n_sample_seq, w.n_kv_heads, w.head_dim)
    st["q"] = synth.queries(w.config, layer, w.n_seq, w.n_q_heads)[:n_sample_seq].numpy()
    return st


def oracle_step(w, st):
    """The same step on the CPU oracle: encode the new token (K, V), write its codes at the
    last position, dense attention over the reconstructed cache."""
    import oracle
    for key in ("k", "v"):
        codes, _, _ = oracle.encode(st[key + "_new"], st[key + "_cb"], w.c, w.b)
        for s, n in enumerate(st["lens"]):
            st[key + "_codes"][s, n - 1] = codes[s]
    return oracle.decode_dense(st["q"], st["k_codes"], st["v_codes"], st["k_cb"], st["v_cb"], st["lens"],
                               w.head_dim ** -0.5, w.c, w.b)


def time_oracle(w, steps, warmup, target_s=None):
    """Times oracle_step on sequence 0 of the batch.  With target_s the step count is chosen so
    that the timed region is about that many seconds of CPU work."""
    import oracle
    st = oracle_sample_state(w, 1)
    for _ in range(warmup):
        oracle_step(w, st)
    if target_s is not None:
        t0 = time.perf_counter()
        oracle_step(w, st)
        one = max(time.perf_counter() - t0, 1e-6)
        steps = int(min(max(target_s / one, 3), 5000))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(w, st)
    dt = (time.perf_counter() - t0) / steps
    toks = int(st["lens"].sum())
    return {"value": toks / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"sequence 0 of the batch, layer 0 ({toks} tokens, all {w.n_kv_heads} KV heads / {w.n_q_heads} query "
                      f"heads): append-encode + dense attention, mean of {steps} steps ({dt * steps:.1f} s); cache encoded "
                      f"by the oracle beforehand (untimed)",
            "ms_per_step": dt * 1e3, "steps": steps}


# ------------------------------------------------------------------------------- extras

def extra_encode_cfg3(cq, dev, reps=5):
    """Prefill encode throughput on config 3 (CQ-2c8b, 8 x 8192 tokens x 32 heads, K and V)."""
    w = synth.WORKLOADS[3]
    D = w.head_dim
    res = {}
    xs, cbs, bufs = [], [], []
    for is_v in (False, True):
        xs.append(synth.layer_activations(w, 0, is_v, w.n_seq, w.n_tokens, device=dev))
        cbs.append(synth.layer_codebooks(w, 0, is_v).to(dev))
        bufs.append(torch.zeros(cq.cq_codes_bytes(w.n_seq, w.n_tokens, w.n_kv_heads, D, w.c, w.b), dtype=torch.uint8,
                                device=dev))
    def run():
        for x, cb, buf in zip(xs, cbs, bufs):
            cq.cq_encode(x, cb, w.c, w.b, buf, w.n_tokens)
    for _ in range(2):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    tokens = w.n_seq * w.n_tokens
    vectors = 2 * tokens * w.n_kv_heads
    res = {"workload": w.name, "ms": ms, "tokens_per_s": tokens / (ms * 1e-3), "vectors_per_s": vectors / (ms * 1e-3),
           "useful_tflops": vectors * 2 * D * (1 << w.b) / (ms * 1e-3) / 1e12,
           "gbs": (vectors * (D * 2 + w.G) + 2 * w.n_kv_heads * D * (1 << w.b) * 4) / (ms * 1e-3) / 1e9}
    # The selection over the 2^b scores of every (vector, group) bounds this kernel: the scores come out of the
    # tensor core into tensor memory, and every one of them has to pass through a min on the ALU pipe, 64 lanes
    # per clock and SM: at least 0.5 operations per score (one 3-input min per two scores).
    pairs = vectors * w.G * (1 << w.b)
    props = torch.cuda.get_device_properties(dev)
    n_sm, mhz = props.multi_processor_count, props.clock_rate / 1e3
    alu_peak = n_sm * 64 * mhz * 1e6
    res["roofline"] = {"bound": "alu", "kernel": "encode_tc_kernel", "achieved": 0.5 * pairs / (ms * 1e-3), "peak": alu_peak,
                       "unit": "lane-ops/s", "frac": 0.5 * pairs / (ms * 1e-3) / alu_peak, "traffic": None,
                       "lane_ops_per_score": 0.5,
                       "peak_source": f"64 ALU lanes/clk/SM x {n_sm} SMs x {mhz:.0f} MHz (device maximum)"}
    attach_traffic(res["roofline"], w.name)
    return res


def extra_learn(cq, dev, iters=100):
    """Centroid learning (Section 3.2.1) on one layer's key tensor of a LLaMA-2-7B-shaped model with the
    paper's calibration size (16 sequences x 2048 tokens): CQ-8c8b, k-means++ and `iters` k-means iterations
    for all 32 heads x 16 groups.  The paper's Table 4 quotes 14 minutes for all 64 (layer, K|V) tensors of
    this model on one A100-40GB: context, another machine."""
    n_vec, n_heads, c, b = 16 * 2048, 32, 8, 8
    w = synth.Workload("learn_llama2_7b_8c8b", 7, c, b, 1, 1, n_heads, n_heads, n_vec)
    x = synth.layer_activations(w, 0, False, 1, n_vec, device=dev)[0].contiguous()
    g = torch.Generator(device="cpu").manual_seed(77)
    u = torch.rand(n_heads, 128 // c, 1 << b, dtype=torch.float64, generator=g).to(dev)
    cq.cq_learn_centroids(x, None, u, c, b, 2)                      # warm-up
    torch.cuda.synchronize()
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record()
    cb0 = cq.cq_kmeanspp_init(x, None, u, c, b)
    e1.record()
    cb, obj = cq.cq_learn_centroids(x, None, u, c, b, iters)
    e2.record()
    torch.cuda.synchronize()
    init_ms, total_ms = e0.elapsed_time(e1), e1.elapsed_time(e2)
    _, obj0 = cq.cq_lloyd_step(x, None, cb0, c, b)
    return {"workload": w.name, "n_vec": n_vec, "problems": n_heads * (128 // c), "iters": iters,
            "init_ms": init_ms, "init_plus_iters_ms": total_ms, "ms_per_iter": (total_ms - init_ms) / iters,
            "objective_init": float(obj0.sum().item()), "objective_final": float(obj.sum().item()),
            "paper_context": "Table 4: 14 min for 64 such tensors (LLaMA-2-7b, CQ-8c8b) on one A100-40GB"}


def extra_encode_wide(cq, dev, w, reps=3):
    """Bulk encode of one tensor of a wide-code workload (chunks of 256 centroids on the tensor cores)."""
    D = w.head_dim
    n_seq = min(w.n_seq, 4)
    x = synth.layer_activations(w, 0, False, n_seq, w.n_tokens, device=dev)
    cb = synth.layer_codebooks(w, 0, False).to(dev)
    buf = torch.zeros(cq.cq_codes_bytes(n_seq, w.n_tokens, w.n_kv_heads, D, w.c, w.b), dtype=torch.uint8, device=dev)
    cq.cq_encode(x, cb, w.c, w.b, buf, w.n_tokens)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        cq.cq_encode(x, cb, w.c, w.b, buf, w.n_tokens)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    vectors = n_seq * w.n_tokens * w.n_kv_heads
    return {"workload": f"{w.name}: {n_seq} x {w.n_tokens} tokens x {w.n_kv_heads} heads, one tensor", "ms": ms,
            "vectors_per_s": vectors / (ms * 1e-3), "useful_tflops": vectors * 2 * D * (1 << w.b) / (ms * 1e-3) / 1e12}


def extra_decode(cq, dev, w, reps=20):
    """One decode-attention call (cq_decode_attn, no append) of another workload, with its roofline."""
    st = DecodeState(w, 0, dev, cq)
    for _ in range(3):
        st.step(cq)
        st.attend(cq)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for e in evs:
        st.attend(cq, e)
    torch.cuda.synchronize()
    ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
    res = {"workload": w.name, "decode_ms": ms, "kv_tokens_per_s": st.kv_tokens() / (ms * 1e-3),
           "query_heads_per_s": w.n_seq * w.n_q_heads / (ms * 1e-3), "roofline": decode_roofline(w, st, ms, dev)}
    attach_traffic(res["roofline"], w.name)
    return res


def extra_prefill(cq, dev, reps=5):
    """cq_prefill_attn on a Mistral-7B-shaped GQA layer (CQ-8c8b): 4 sequences whose caches hold 8192 tokens,
    the newest 2048 of which are the chunk being prefilled (causal)."""
    w0 = synth.WORKLOADS[2]
    n_seq, cap, n_q = 4, 8192, 2048
    w = synth.Workload("prefill_mistral_7b_gqa_8c8b_chunk2048_of_8192", 8, w0.c, w0.b, 1, n_seq, w0.n_q_heads, w0.n_kv_heads, cap)
    st = DecodeState(w, 0, dev, cq)
    g = torch.Generator(device="cpu").manual_seed(88)
    q = torch.randn(n_seq, n_q, w.n_q_heads, w.head_dim, generator=g).to(torch.float16).to(dev)
    out = torch.empty(n_seq, n_q, w.n_q_heads, w.head_dim, dtype=torch.float32, device=dev)
    run = lambda: cq.cq_prefill_attn(q, st.k_codes, st.v_codes, st.k_cb, st.v_cb, st.seq_lens, st.scale, w.c, w.b, cap, out=out)
    for _ in range(2):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    # useful contraction work: every (query, head) against the tokens up to its position, QK^T and PV
    keys = sum(cap - n_q + i + 1 for i in range(n_q))
    flops = 4.0 * n_seq * w.n_q_heads * keys * w.head_dim
    peak = None
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
    except Exception:
        peak = 1590.0
    tf = flops / (ms * 1e-3) / 1e12
    res = {"workload": w.name, "ms": ms, "query_tokens_per_s": n_seq * n_q / (ms * 1e-3),
           "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "traffic": None,
                        "peak_source": "measured bf16 GEMM burst (fp16 has the same nominal rate); mma.sync path"}}
    attach_traffic(res["roofline"], w.name)
    return res


def extra_decode_rope(cq, dev, w, reps=5):
    """Attention over codes of pre-RoPE keys (cq_decode_attn_rope: the tuned kernel where the shape has one) on the
    shape of a decode workload."""
    st = DecodeState(w, 0, dev, cq)
    P = w.head_dim // 2
    ang = torch.arange(st.cap, dtype=torch.float64, device=dev)[:, None] * \
        (10000.0 ** (-torch.arange(P, dtype=torch.float64, device=dev) / P))[None, :]
    cs, sn = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    run = lambda: cq.cq_decode_attn_rope(st.q, st.k_codes, st.v_codes, st.k_cb, st.v_cb, st.seq_lens, cs, sn, st.scale,
                                         w.c, w.b, st.cap, out=st.out, workspace=st.ws)
    for _ in range(2):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    hbm, _ = measured_peaks()
    gbs = (st.algorithmic_bytes() + 2 * cs.numel() * 4) / (ms * 1e-3) / 1e9
    return {"workload": w.name + " with pre-RoPE key codes", "decode_ms": ms, "kv_tokens_per_s": st.kv_tokens() / (ms * 1e-3),
            "gbs": gbs, "frac_of_measured_hbm": gbs / hbm}


# --------------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg0", "cfg1", "cfg2", "cfg4"])
    ap.add_argument("--extras", default="default", choices=["none", "default", "decode", "all"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    w = synth.WORKLOADS[int(args.workload[3])]
    config = {"workload": w.name, "c": w.c, "b": w.b, "n_seq": w.n_seq, "n_q_heads": w.n_q_heads,
              "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "context": w.n_tokens, "layers_per_step": w.n_layers,
              "step": "append-encode new token (K,V) + decode attention",
              "l2": "inputs exceed L2 (code buffers > 126 MB)" if w.name.startswith(("cfg2", "cfg4")) else
                    "inputs fit L2 (small case)"}

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if rank != 0:
            return 0
        steps = max(1, min(args.steps, 20))
        r = time_oracle(w, steps, max(1, min(args.warmup, 2)))
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": steps, "warmup": max(1, min(args.warmup, 2)), "ms_per_step": r["ms_per_step"],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": config,
                "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
                "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py --impl ours needs a CUDA device: the library has no CPU fallback")
    import paper_2405_03917_b200 as cq
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)

    states = [DecodeState(w, layer, dev, cq) for layer in range(w.n_layers)]
    st = states[0]
    torch.cuda.synchronize()

    def step(ev):
        # the events bracket the decode-attention call of the last layer
        for i, sti in enumerate(states):
            sti.step(cq, ev if (ev is not None and i == len(states) - 1) else None)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    total_ms, inner_ms = time_steps(step, args.steps, args.warmup, world, dev)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = total_ms / args.steps
    kv_tokens = sum(x.kv_tokens() for x in states) * world
    value = kv_tokens / (ms_per_step * 1e-3)

    # end to end: host buffers in, host result out, through cq_decode_step_host
    D = w.head_dim
    ws_h = torch.empty(cq.cq_decode_step_host_workspace_bytes(w.n_seq, w.n_q_heads, w.n_kv_heads, D, w.c, w.b, st.cap),
                       dtype=torch.uint8, device=dev)
    def pinned_block(x):
        # query, key and value of a step back to back in one pinned block: they travel in one copy
        parts = (x.q, x.k_new, x.v_new)
        block = torch.empty(sum(p.numel() for p in parts), dtype=torch.float16).pin_memory()
        views, at = [], 0
        for p in parts:
            v = block[at:at + p.numel()].view(p.shape)
            v.copy_(p.cpu())
            views.append(v)
            at += p.numel()
        return tuple(views)
    host = [pinned_block(x) for x in states]
    lens_h = (st.lens_cpu - 1).contiguous()
    out_h = torch.empty(w.n_seq, w.n_q_heads, D, dtype=torch.float32).pin_memory()

    def e2e_step():
        for x, (q_h, k_h, v_h) in zip(states, host):
            cq.cq_decode_step_host(q_h, k_h, v_h, lens_h, x.k_codes, x.v_codes, x.k_cb, x.v_cb, x.scale, w.c, w.b,
                                   x.cap, out_h, ws_h)
    for _ in range(3):
        e2e_step()
    torch.cuda.synchronize()
    barrier(world)
    t0 = time.perf_counter()
    n_e2e = max(5, args.steps // 2)
    for _ in range(n_e2e):
        e2e_step()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / n_e2e, world, dev)
    q_h, k_h, v_h = host[0]
    h2d = len(states) * (q_h.numel() * 2 + k_h.numel() * 2 + v_h.numel() * 2 + lens_h.numel() * 4)
    d2h = len(states) * out_h.numel() * 4

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return 0

    last = states[-1]
    dec_ms = statistics.mean(inner_ms)
    roofline = decode_roofline(w, last, dec_ms, dev, (clocks or {}).get("sm_mhz"))
    attach_traffic(roofline, w.name)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "query_heads_per_s": w.n_seq * w.n_q_heads * len(states) * world / (ms_per_step * 1e-3),
            "clocks": clocks,
            "e2e": {"value": kv_tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            # per layer: attention (which appends the new token where the kernel can) and merge, else also the append-encode
            "gpu_launches": args.steps * len(states) * (st.fused_launches if st.fused_launches <= 2 else 3),
            "roofline": roofline}

    if args.extras != "none" and world == 1:
        extras = {}
        try:
            del st, states, last
            torch.cuda.empty_cache()
            if args.extras != "decode":
                extras["encode"] = extra_encode_cfg3(cq, dev)
            # the other decode workloads, each with its own roofline object (one layer each)
            extras["decode_cfg1"] = extra_decode(cq, dev, synth.WORKLOADS[1])
            extras["decode_cfg4_layer0"] = extra_decode(cq, dev, synth.WORKLOADS[4])
            extras["decode_cfg5_8c10b"] = extra_decode(cq, dev, synth.WORKLOADS[5], reps=5)
            extras["decode_cfg6_2c8b"] = extra_decode(cq, dev, synth.WORKLOADS[6])
            extras["prefill"] = extra_prefill(cq, dev)
            extras["decode_rope_cfg1"] = extra_decode_rope(cq, dev, synth.WORKLOADS[1])
            if args.extras in ("decode", "all"):
                extras["encode_cfg5_8c10b"] = extra_encode_wide(cq, dev, synth.WORKLOADS[5])
            if args.extras == "all":
                extras["learn"] = extra_learn(cq, dev)
        except Exception as e:      # extras never hide the headline number
            extras["error"] = repr(e)
        line["extras"] = extras
    if not args.no_cpu_baseline and world == 1:
        st = states = last = None
        torch.cuda.empty_cache()
        r = time_oracle(w, 10, 1, target_s=12.0)
        line["cpu_baseline"] = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
