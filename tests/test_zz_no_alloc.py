"""bs_softmax_verify_noalloc against bs_softmax_verify, through the C ABI.

Some users of the library cannot allocate device memory at the call site: a serving loop that
lives inside a memory pool fixed at start-up, a plugin that is only handed its input and output
buffers, a path where cudaMalloc is banned because it stalls the whole device.  For them the
library carries its own scratch array; this test checks that the variant using it gives exactly
what the workspace variant gives, twice in a row (the array keeps the previous call's contents),
and that it refuses sizes the array cannot hold.

The file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from paper_2505_15141_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(seed, B, G, V, dtype):
    g = torch.Generator(device="cpu"); g.manual_seed(seed)
    t = (torch.randn(B, G + 1, V, generator=g) * 3).to(dtype).to(DEV)
    d = (t[:, :G].float().cpu() + torch.randn(B, G, V, generator=g)).to(dtype).to(DEV)
    rng = np.random.default_rng(seed)
    gamma = torch.as_tensor(rng.integers(0, G + 1, size=B).astype(np.int32), device=DEV)
    u = torch.as_tensor(rng.random((B, G)).astype(np.float32) * 0.998 + 0.001, device=DEV)
    tok = wl.draw_draft_tokens(d, 1.0, rng.random((B, G)).astype(np.float32) * 0.998 + 0.001).contiguous()
    return t, d, tok, gamma, u


def _run(fn, t, d, tok, gamma, u, T, **kw):
    B, G1, V = t.shape
    acc = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    p = torch.full((B, G1 - 1), -1.0, dtype=torch.float32, device=DEV)
    q = torch.full((B, G1 - 1), -1.0, dtype=torch.float32, device=DEV)
    fn(t, d, tok, gamma, u, T, acc, p, q, **kw)
    torch.cuda.synchronize()
    return acc, p, q


@pytest.mark.parametrize("dtype,V", [(torch.float32, 20000), (torch.bfloat16, 32000), (torch.float32, 1001)])
def test_noalloc_matches_workspace_variant_twice(lib, dtype, V):
    B, G = 12, 5
    ws = lib.new_workspace(B, G, V, DEV)
    for call, (seed, T) in enumerate([(100 + V, 1.0), (200 + V, 0.7)]):      # two calls in a row, new inputs
        t, d, tok, gamma, u = _inputs(seed, B, G, V, dtype)
        want = _run(lib.bs_softmax_verify, t, d, tok, gamma, u, T, workspace=ws)
        got = _run(lib.bs_softmax_verify_noalloc, t, d, tok, gamma, u, T)
        assert torch.equal(got[0], want[0]), f"call {call}: accept_len differs"
        # same kernels, same order of operations: the tolerance of the parity tests (1e-5) is met exactly
        assert torch.allclose(got[1], want[1], atol=1e-5, rtol=0) and torch.allclose(got[2], want[2], atol=1e-5, rtol=0)
        assert torch.equal(got[1], want[1]) and torch.equal(got[2], want[2])
    # greedy mode on the same array
    t, d, tok, gamma, u = _inputs(7, B, G, V, dtype)
    tok = t[:, :G].float().argmax(-1).to(torch.int32).contiguous()
    want = _run(lib.bs_softmax_verify, t, None, tok, gamma, None, 0.0, workspace=ws)
    got = _run(lib.bs_softmax_verify_noalloc, t, None, tok, gamma, None, 0.0)
    assert torch.equal(got[0], want[0]) and torch.equal(got[0].cpu(), gamma.cpu())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_noalloc_matches_the_oracle(lib, dtype):
    """The entry point by itself against the CPU checker (Algorithm 6's accept loop): accepted lengths
    exact except at flagged near-ties of the accept test, token probabilities within 1e-5.  One
    sequence carries a token outside the vocabulary: that position counts as rejected, as the header
    says, although no status word can be read back from the built-in scratch."""
    from oracle import verify as ov
    B, G, V, T = 9, 4, 32000, 0.9
    t, d, tok, gamma, u = _inputs(31 + (dtype == torch.bfloat16), B, G, V, dtype)
    gamma = torch.full_like(gamma, G)
    tok[4, 1] = V + 3
    acc, p, q = _run(lib.bs_softmax_verify_noalloc, t, d, tok, gamma, u, T)
    flagged = 0
    for b in range(B):
        toks = tok[b].cpu().numpy().copy()
        cut = G
        if b == 4:
            toks[1], cut = 0, 1                                  # the oracle sees valid positions only
        ref = ov.verify_sequence(t[b].float().cpu().numpy(), d[b].float().cpu().numpy(), toks, cut,
                                 u[b].cpu().numpy(), 0.5, T)
        got = int(acc[b])
        if got != ref.tau:
            j = min(got, ref.tau)
            assert abs(ref.accept_margin[j]) < ov.ACCEPT_TIE, (b, got, ref.tau)
            flagged += 1
        assert got <= cut
        assert np.abs(p[b, :cut].cpu().numpy() - ref.p_tok).max() <= 1e-5
        assert np.abs(q[b, :cut].cpu().numpy() - ref.q_tok).max() <= 1e-5
    assert flagged <= 1


def test_noalloc_rejects_sizes_beyond_its_scratch(lib):
    B, G, V = 512, 8, 152064
    assert lib.bs_workspace_bytes(B, G, V) > lib.BS_NOALLOC_SCRATCH_BYTES
    # refused on the host before anything is read or launched: the pointers are never touched
    code = lib._lib.bs_softmax_verify_noalloc(None, None, lib.BS_F32, None, None, None, 1.0, B, G, V,
                                              None, None, None, None)
    assert code == lib.BS_ERR_WORKSPACE
    assert lib.bs_workspace_bytes(256, 8, 152064) <= lib.BS_NOALLOC_SCRATCH_BYTES
