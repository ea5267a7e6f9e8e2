"""CPU oracle (fp64) for the trimmed-vocabulary draft head.  TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy wrapper around ``vt_oracle.c``; it exists so tests, the smoke
check and the bench's CPU-baseline leg can call the oracle.  The CUDA library and
its Python binding never import this package, and this package never imports them.
"""
from .vt_oracle import (build, num_threads, bf16_to_f64, compact, logits, log_softmax, topk, remap,
                        coverage, draft_head)

__all__ = ["build", "num_threads", "bf16_to_f64", "compact", "logits", "log_softmax", "topk", "remap",
           "coverage", "draft_head"]
