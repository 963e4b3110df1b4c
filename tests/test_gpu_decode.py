"""GPU parity of the decoding step (dma_delta_range + dma_decode) against the oracle: selected key sets bit-exact,
outputs within the element type's tolerance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, bits_equal, oracle_mask

pytestmark = pytest.mark.gpu


def run_case(case, cap_extra=0, seed=21, tie_heads=False):
    """The case's K, V (and W_delta, A) form the cache; the query of every head is a fresh N(0,1) vector."""
    inp = wl.make_inputs(case)
    dev = torch.device("cuda:0")
    B, N, Hq, Hkv, d = case.B, case.L, case.Hq, case.Hkv, case.d
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, d, generator=g).to(case.torch_dtype)
    cap = N + cap_extra
    Kc = torch.zeros(B, cap, Hkv, d, dtype=case.torch_dtype); Kc[:, :N] = inp["K"]
    Vc = torch.zeros(B, cap, Hkv, d, dtype=case.torch_dtype); Vc[:, :N] = inp["V"]
    A = inp["A"].clone()
    if tie_heads:
        A[0] = 0.0                                   # delta == 1 for every key of head 0: the w lowest indices win
    p = dma.problem(B, Hq, Hkv, N, d, case.w, dtype=case.torch_dtype)
    p.k_stride[0], p.k_stride[1], p.k_stride[2] = cap * Hkv * d, Hkv * d, d
    p.v_stride[0], p.v_stride[1], p.v_stride[2] = cap * Hkv * d, Hkv * d, d
    Kd, Vd = Kc.to(dev), Vc.to(dev)
    delta = torch.full((B, Hq, cap), -1.0, device=dev)
    # the cache is filled in two appends, as a prefill followed by decoding steps would do
    half = N // 2
    dma.dma_delta_range(p, Vd, inp["W_delta"].to(dev), A.to(dev), delta, 0, half)
    dma.dma_delta_range(p, Vd, inp["W_delta"].to(dev), A.to(dev), delta, half, N)
    o, lse, idx = dma.dma_decode(p, q.to(dev), Kd, Vd, delta, want_idx=True)
    torch.cuda.synchronize()
    # oracle: delta in the pinned fp32 arithmetic, then the definition
    z, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), A.numpy(), Hq)
    assert bits_equal(delta[:, :, :N], dl), "delta cache differs from the pinned arithmetic"
    assert (delta[:, :, N:] == -1.0).all(), "entries beyond the appended range were touched"
    ro, rl, ridx = oracle.decode(q.double().numpy(), inp["K"].double().numpy(), inp["V"].double().numpy(), dl, case.w)
    assert np.array_equal(idx.cpu().numpy(), ridx), "selected key sets differ"
    assert_close(o, ro, case.dtype, f"{case.name}: o")
    assert_close(lse, rl, case.dtype, f"{case.name}: lse", lse=True)


@pytest.mark.parametrize("kw", [
    dict(B=1, Hq=2, Hkv=2, L=256, d=64, w=64, dtype="fp32"),
    dict(B=2, Hq=4, Hkv=2, L=1000, d=64, w=100, dtype="bf16"),
    dict(B=2, Hq=8, Hkv=2, L=3001, d=128, w=512, dtype="bf16"),       # ragged: two splits, the second partly empty
    dict(B=1, Hq=4, Hkv=4, L=5000, d=128, w=1, dtype="fp32"),         # a single key
    dict(B=1, Hq=4, Hkv=1, L=700, d=128, w=4096, dtype="bf16"),       # w >= N: dense attention over the cache
])
def test_small_cases(kw):
    run_case(wl.small(wl.CONFIGS["2"], name="decode-small", backward=False, **kw), cap_extra=37)


def test_ties_go_to_the_lower_index():
    run_case(wl.small(wl.CONFIGS["2"], name="decode-ties", backward=False, B=1, Hq=2, Hkv=1, L=4500, d=128, w=300), tie_heads=True)


def test_long_cache_config5_shapes():
    # the paper's decode setting on the long-context shapes: 65 536 cached keys, w = 4096, 32 / 8 heads
    run_case(wl.CONFIGS["5"], cap_extra=128)
