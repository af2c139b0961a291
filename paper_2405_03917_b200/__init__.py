"""B200-native Coupled Quantization (CQ) KV-cache hot path: `cq_encode` and `cq_decode_attn`.

The work is done by hand-written sm_100a CUDA kernels in `libcq.so` (built in-tree by
`paper_2405_03917_b200.build`), reached through the C ABI declared in `include/cq.h`.
This package only marshals torch tensors into that ABI; there is no CPU or PyTorch
fallback, and importing `binding` fails loudly when the library is missing.
"""
from .binding import (CQError, lib, library_path, cq_layout_version, cq_status_string, cq_codes_bytes, cq_encode,
                      cq_codes_to_rowmajor, cq_codes_from_rowmajor, cq_decode_attn_workspace_bytes, cq_decode_attn, cq_decode_attn_rope, cq_prefill_attn, cq_encode_kv, cq_decode_attn_static,
                      cq_decode_step_workspace_bytes, cq_decode_step_launches, cq_decode_step, cq_decode_step_host_workspace_bytes, cq_decode_step_host,
                      cq_learn_workspace_bytes,
                      cq_kmeanspp_init, cq_lloyd_step, cq_learn_centroids, EXPORTS)

__all__ = ["CQError", "lib", "library_path", "cq_layout_version", "cq_status_string", "cq_codes_bytes", "cq_encode",
           "cq_codes_to_rowmajor", "cq_codes_from_rowmajor", "cq_decode_attn_workspace_bytes", "cq_decode_attn", "cq_decode_attn_rope", "cq_prefill_attn", "cq_encode_kv", "cq_decode_attn_static",
           "cq_decode_step_workspace_bytes", "cq_decode_step_launches", "cq_decode_step", "cq_decode_step_host_workspace_bytes", "cq_decode_step_host",
           "cq_learn_workspace_bytes", "cq_kmeanspp_init",
           "cq_lloyd_step", "cq_learn_centroids", "EXPORTS"]
