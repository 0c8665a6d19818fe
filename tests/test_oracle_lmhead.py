"""Pin of the LM-head checker: the library matmul against the written-out triple loop."""
import numpy as np

from oracle.lmhead import lmhead_logits


def test_lmhead_matches_triple_loop():
    rng = np.random.default_rng(0)
    H = rng.normal(size=(3, 5)).astype(np.float32)
    W = rng.normal(size=(5, 4)).astype(np.float32)
    want = np.zeros((3, 4))
    for r in range(3):
        for v in range(4):
            for k in range(5):
                want[r, v] += float(H[r, k]) * float(W[k, v])
    got = lmhead_logits(H, W)
    assert got.dtype == np.float64 and np.allclose(got, want, atol=1e-14)
    # not the transposed product
    assert not np.allclose(lmhead_logits(H, W), lmhead_logits(H[:, ::-1], W))
