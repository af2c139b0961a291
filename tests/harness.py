"""Shared helpers of the parity tests: acceptance rules and case builders.

Acceptance rules (written here once, used by every parity test):
  * codes: bit-exact against the oracle, except where the oracle's distance of the
    CUDA code exceeds the oracle's best distance by less than 1e-4 relative
    (d_gpu - d_best < 1e-4 * d_gpu); those near-ties are accepted and counted;
  * attention: max-abs error <= 2e-3 and relative L2 error <= 1e-3 against the oracle.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2405_03917_b200 import synth

CODE_TIE_REL = 1e-4
ATTN_MAX_ABS = 2e-3
ATTN_REL_L2 = 1e-3


def check_codes(x_np, cb_np, gpu_codes, c, b, oracle_result=None):
    """x_np fp16 (n_vec, n_heads, D); gpu_codes integer (n_vec, n_heads, G).
    Returns (n_near_ties, n_total); raises AssertionError on a real mismatch."""
    codes, d_best, _ = oracle_result if oracle_result is not None else oracle.encode(x_np, cb_np, c, b)
    gpu_codes = np.asarray(gpu_codes).astype(np.int32)
    assert gpu_codes.shape == codes.shape
    assert gpu_codes.min() >= 0 and gpu_codes.max() < (1 << b)
    diff = gpu_codes != codes
    n_diff = int(diff.sum())
    if n_diff:
        d_gpu = oracle.code_distance(x_np, cb_np, gpu_codes, c, b)
        ok = (d_gpu - d_best) < CODE_TIE_REL * d_gpu
        ok |= (d_gpu == d_best)                      # exact ties, including 0 == 0
        bad = diff & ~ok
        assert not bad.any(), (
            f"{int(bad.sum())} codes differ outside the near-tie band; first at {np.argwhere(bad)[0].tolist()}: "
            f"gpu {gpu_codes[bad][0]} (d={d_gpu[bad][0]:.9g}) oracle {codes[bad][0]} (d={d_best[bad][0]:.9g})")
    return n_diff, int(codes.size)


def attn_errors(out_gpu, out_ref):
    out_gpu = np.asarray(out_gpu, dtype=np.float64)
    out_ref = np.asarray(out_ref, dtype=np.float64)
    assert np.isfinite(out_gpu).all(), "non-finite attention output"
    max_abs = float(np.abs(out_gpu - out_ref).max()) if out_ref.size else 0.0
    denom = float(np.sqrt((out_ref ** 2).sum()))
    rel = float(np.sqrt(((out_gpu - out_ref) ** 2).sum()) / denom) if denom > 0 else max_abs
    return max_abs, rel


def check_attn(out_gpu, out_ref, what=""):
    max_abs, rel = attn_errors(out_gpu, out_ref)
    assert max_abs <= ATTN_MAX_ABS, f"{what}: max-abs error {max_abs:.3e} > {ATTN_MAX_ABS}"
    assert rel <= ATTN_REL_L2, f"{what}: relative L2 error {rel:.3e} > {ATTN_REL_L2}"
    return max_abs, rel


def small_workload(name, config, c, b, n_seq, n_q_heads, n_kv_heads, n_tokens, head_dim=128):
    return synth.Workload(name, config, c, b, 1, n_seq, n_q_heads, n_kv_heads, n_tokens, head_dim=head_dim)


def generic_case(seed, n_seq, n_tokens, n_q_heads, n_kv_heads, head_dim, c, b, outliers=True):
    """Random inputs for shapes the config generator does not cover (head_dim != 128):
    same recipe in miniature (low-rank plus noise, a few shifted key channels)."""
    g = torch.Generator().manual_seed(seed)
    rank = max(2, head_dim // 4)
    def acts(n, shift):
        A = torch.randn(n_kv_heads, head_dim, rank, generator=g) / rank ** 0.5
        mu = 0.5 * torch.randn(n_kv_heads, head_dim, generator=g)
        z = torch.randn(n, n_kv_heads, rank, generator=g)
        x = torch.einsum("nhr,hdr->nhd", z, A) + mu + 0.1 * torch.randn(n, n_kv_heads, head_dim, generator=g)
        if shift:
            x[:, :, :: max(1, head_dim // 3)] = 8 + 5 * x[:, :, :: max(1, head_dim // 3)]
        return x.contiguous()
    K = 1 << b
    G = head_dim // c
    xk = acts(n_seq * n_tokens, outliers).view(n_seq, n_tokens, n_kv_heads, head_dim).to(torch.float16).contiguous()
    xv = acts(n_seq * n_tokens, False).view(n_seq, n_tokens, n_kv_heads, head_dim).to(torch.float16).contiguous()
    kcb = acts(K, outliers).view(K, n_kv_heads, G, c).permute(1, 2, 0, 3).contiguous()
    vcb = acts(K, False).view(K, n_kv_heads, G, c).permute(1, 2, 0, 3).contiguous()
    q = torch.randn(n_seq, n_q_heads, head_dim, generator=g).to(torch.float16)
    return xk, xv, kcb, vcb, q


def oracle_encode_rowmajor(x, cb, c, b):
    """x torch fp16 (n_seq, n_tokens, n_heads, D) on any device -> int32 numpy codes
    (n_seq, n_tokens, n_heads, G) plus the oracle's (codes, d_best, d_second) triple."""
    xn = x.detach().cpu().numpy()
    n_seq, n_tokens, n_heads, D = xn.shape
    res = oracle.encode(xn.reshape(n_seq * n_tokens, n_heads, D), cb.detach().cpu().numpy(), c, b)
    return res[0].reshape(n_seq, n_tokens, n_heads, D // c), res
