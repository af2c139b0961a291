"""CPU oracle for the CQ hot path -- test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline legs may
import this package; the CUDA library and its Python binding never do.
"""
from .cq_oracle import (build, encode, code_distance, dequant, decode_dense, decode_dense_rope, decode_lut, prefill_dense,
                        kmeanspp_init, lloyd_step, num_threads, set_num_threads)

__all__ = ["build", "encode", "code_distance", "dequant", "decode_dense", "decode_dense_rope", "decode_lut", "prefill_dense", "kmeanspp_init", "lloyd_step",
           "num_threads", "set_num_threads"]
