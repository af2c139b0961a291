"""Seeded synthetic inputs for the CQ hot path.

This module only draws random numbers and shapes them like LLM key/value
activations; it holds none of the method's arithmetic (no distances, no
argmin, no attention).  Both the CUDA path and the CPU oracle read the
tensors produced here, so neither ever consumes the other's output.

Recipe (one `HeadSource` per (config, layer, KV head, K|V)):

* mixing matrix ``A`` of shape (128, 32) with entries N(0, 1)/sqrt(32),
  channel offsets ``mu`` with entries N(0, sigma=0.5);
* a token is ``x = A z + mu + 0.1 eps`` with ``z ~ N(0, I_32)`` and
  ``eps ~ N(0, I_128)``: strongly inter-dependent, low-rank channels, the
  structure the paper reports for real K/V activations (Section 3.1);
* keys only: 4 distinct outlier channels per head, transformed as
  ``x_ch <- mu_ch + 8 + 5 (x_ch - mu_ch)`` (mean +8, std x5), the outlier
  key channels the paper mentions in Sections 2.3 and 3.2;
* activations are cast to fp16; codebooks are 256 further fp32 draws from
  the same source, centroid j of group g being channels [g c, (g+1) c) of
  draw j;
* queries are fp16 N(0, 1).

The small per-head parameters (A, mu, outlier channels) always come from a
CPU generator, so they are identical whichever device draws the tokens.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch

HEAD_DIM = 128
LATENT = 32
N_OUTLIER = 4
NOISE = 0.1


def head_seed(config: int, layer: int, head: int, is_v: bool) -> int:
    return 1_000_000 * config + 1_000 * layer + 2 * head + (1 if is_v else 0)


@dataclasses.dataclass
class HeadSource:
    seed: int
    is_v: bool
    A: torch.Tensor          # (128, 32) fp32, CPU
    mu: torch.Tensor         # (128,) fp32, CPU
    outliers: torch.Tensor   # (4,) int64, CPU (empty for V)

    def _params(self, device):
        return self.A.to(device), self.mu.to(device), self.outliers.to(device)

    def draw(self, n: int, stream: int, device="cpu") -> torch.Tensor:
        """n fp32 vectors (n, 128).  `stream` separates independent draws
        (0 = codebook parents, 1 = activations, 2.. = extra)."""
        g = torch.Generator(device=device)
        g.manual_seed(self.seed * 16 + stream + 12345)
        A, mu, out = self._params(device)
        z = torch.randn(n, LATENT, generator=g, device=device, dtype=torch.float32)
        eps = torch.randn(n, HEAD_DIM, generator=g, device=device, dtype=torch.float32)
        x = z @ A.t() + mu + NOISE * eps
        if out.numel():
            x[:, out] = mu[out] + 8.0 + 5.0 * (x[:, out] - mu[out])
        return x

    def activations(self, n: int, device="cpu", stream: int = 1) -> torch.Tensor:
        """n fp16 token vectors (n, 128)."""
        return self.draw(n, stream, device).to(torch.float16)

    def codebook(self, c: int, b: int, device="cpu") -> torch.Tensor:
        """fp32 codebook (G, 2^b, c): centroid j of group g = channels of parent draw j."""
        k = 1 << b
        parents = self.draw(k, 0, device)                  # (K, 128) fp32
        G = HEAD_DIM // c
        return parents.view(k, G, c).permute(1, 0, 2).contiguous()


def head_source(config: int, layer: int, head: int, is_v: bool) -> HeadSource:
    seed = head_seed(config, layer, head, is_v)
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    A = torch.randn(HEAD_DIM, LATENT, generator=g, dtype=torch.float32) / (LATENT ** 0.5)
    mu = 0.5 * torch.randn(HEAD_DIM, generator=g, dtype=torch.float32)
    if is_v:
        outliers = torch.empty(0, dtype=torch.int64)
    else:
        outliers = torch.randperm(HEAD_DIM, generator=g)[:N_OUTLIER].sort().values
    return HeadSource(seed=seed, is_v=is_v, A=A, mu=mu, outliers=outliers)


def queries(config: int, layer: int, n_seq: int, n_q_heads: int, device="cpu") -> torch.Tensor:
    """fp16 N(0,1) queries (n_seq, n_q_heads, 128)."""
    g = torch.Generator(device=device)
    g.manual_seed(7_000_000_000 + 1_000_000 * config + layer)
    return torch.randn(n_seq, n_q_heads, HEAD_DIM, generator=g, device=device,
                       dtype=torch.float32).to(torch.float16)


def seq_lens_uniform(config: int, n_seq: int, lo: int, hi: int) -> torch.Tensor:
    """int32 lengths uniform in [lo, hi], seeded (CPU)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(9_000_000_000 + config)
    return torch.randint(lo, hi + 1, (n_seq,), generator=g, dtype=torch.int64).to(torch.int32)


@dataclasses.dataclass
class Workload:
    """Shapes of one benchmark configuration."""
    name: str
    config: int
    c: int
    b: int
    n_layers: int
    n_seq: int
    n_q_heads: int
    n_kv_heads: int
    n_tokens: int                 # context per sequence (max for varlen)
    min_tokens: Optional[int] = None   # set => lengths uniform in [min_tokens, n_tokens]
    head_dim: int = HEAD_DIM

    @property
    def G(self) -> int:
        return self.head_dim // self.c

    def lengths(self) -> torch.Tensor:
        if self.min_tokens is None:
            return torch.full((self.n_seq,), self.n_tokens, dtype=torch.int32)
        return seq_lens_uniform(self.config, self.n_seq, self.min_tokens, self.n_tokens)


WORKLOADS: List[Workload] = [
    Workload("cfg0_tiny_8c8b", 0, 8, 8, 1, 1, 1, 1, 1024),
    Workload("cfg1_llama2_7b_4c8b_decode", 1, 4, 8, 1, 16, 32, 32, 4096),
    Workload("cfg2_mistral_7b_gqa_8c8b_decode", 2, 8, 8, 1, 64, 32, 8, 16384),
    Workload("cfg3_2c8b_prefill_encode", 3, 2, 8, 1, 8, 32, 32, 8192),
    Workload("cfg4_llama2_13b_8c8b_full_step", 4, 8, 8, 40, 32, 40, 40, 32768, min_tokens=8192),
    # CQ-8c10b (1024 centroids per group, 1.25 bytes per code), Llama-2-7B-shaped heads; not one of the
    # measured configurations of the headline metric: a workload for the wide-code path
    Workload("cfg5_llama2_7b_8c10b_decode", 5, 8, 10, 1, 16, 32, 32, 8192),
    # CQ-2c8b (64 groups, 4 bits per channel) decode on config 1's shape: the workload of the 64-group decode kernel
    Workload("cfg6_llama2_7b_2c8b_decode", 6, 2, 8, 1, 16, 32, 32, 4096),
]


def layer_codebooks(w: Workload, layer: int, is_v: bool, device="cpu") -> torch.Tensor:
    """fp32 codebooks (n_kv_heads, G, 2^b, c) of one layer."""
    return torch.stack([head_source(w.config, layer, h, is_v).codebook(w.c, w.b, device)
                        for h in range(w.n_kv_heads)])


def layer_activations(w: Workload, layer: int, is_v: bool, n_seq: int, n_tokens: int,
                      device="cpu", heads: Optional[List[int]] = None) -> torch.Tensor:
    """fp16 activations (n_seq, n_tokens, n_heads, 128) of one layer; head h of the
    result is the (n_seq * n_tokens) draw of that head's source reshaped, so any
    (sequence, head) slice can be regenerated alone with the same arguments."""
    heads = list(range(w.n_kv_heads)) if heads is None else heads
    out = torch.empty(n_seq, n_tokens, len(heads), w.head_dim, dtype=torch.float16, device=device)
    for i, h in enumerate(heads):
        src = head_source(w.config, layer, h, is_v)
        out[:, :, i, :] = src.activations(n_seq * n_tokens, device).view(n_seq, n_tokens, w.head_dim)
    return out
