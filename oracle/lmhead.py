"""CPU checker for the LM-head projection that precedes verification.  TEST INFRASTRUCTURE.

Algorithm 6 (second line) evaluates the target model on all drafted positions
in parallel; the last step of that evaluation is logits = H W with H the final
hidden states [rows, d] and W the output embedding [d, V].  The checker is the
textbook product in fp64 on exactly the bf16 values the GPU reads (bf16 -> fp64
is exact).  Pin: numpy.matmul is the library routine; tests compare it with an
explicit triple loop on a tiny case.
"""
from __future__ import annotations

import numpy as np


def lmhead_logits(H: np.ndarray, W: np.ndarray) -> np.ndarray:
    """logits[r, v] = sum_k H[r, k] W[k, v], fp64."""
    return np.asarray(H, dtype=np.float64) @ np.asarray(W, dtype=np.float64)
