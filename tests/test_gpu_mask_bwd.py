"""GPU parity of dma_mask_bwd (mask-generation backward, Sec. 4.3 / Eq. delta_calc differentiated) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, problem_of

pytestmark = pytest.mark.gpu


def run_case(case, seed):
    inp = wl.make_inputs(case)
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(seed)
    dM = torch.randn(case.B, case.Hq, case.L, generator=g)
    dV0 = torch.randn(case.B, case.L, case.Hkv, case.d, generator=g).to(case.torch_dtype)
    p = problem_of(case)
    V, W, A = inp["V"].to(dev), inp["W_delta"].to(dev), inp["A"].to(dev)
    bias, _, _ = dma.dma_mask_build(p, V, W, A)
    dV = dV0.to(dev).clone()
    _, dW, dA = dma.dma_mask_bwd(p, V, W, A, bias, dM.to(dev), dV)
    torch.cuda.synchronize()
    rV, rW, rA = oracle.mask_backward(inp["V"].double().numpy(), inp["W_delta"].double().numpy(), inp["A"].double().numpy(),
                                      dM.double().numpy(), case.Hq)
    assert_close(dV, dV0.double().numpy() + rV, case.dtype, f"{case.name}: dV (in/out)")
    assert_close(dW, rW, "fp32", f"{case.name}: dW_delta")
    assert_close(dA, rA, "fp32", f"{case.name}: dA")
    return p, V, W, A, bias, dM.to(dev), dV0.to(dev)


@pytest.mark.parametrize("kw", [
    dict(B=1, Hq=2, Hkv=2, L=256, d=64, w=64, dtype="fp32"),
    dict(B=2, Hq=4, Hkv=2, L=300, d=64, w=64, dtype="bf16"),          # ragged tail, GQA, d = 64
    dict(B=2, Hq=8, Hkv=2, L=517, d=128, w=128, dtype="bf16"),        # ragged tail, G = 4
    dict(B=1, Hq=4, Hkv=4, L=1024, d=128, w=256, dtype="fp32"),
    dict(B=1, Hq=16, Hkv=1, L=130, d=128, w=32, dtype="bf16"),        # G = 16 (largest supported group)
])
def test_small_cases(kw):
    run_case(wl.small(wl.CONFIGS["2"], name="mask-bwd-small", backward=True, **kw), seed=11)


def test_full_size_config3_and_reproducible():
    case = wl.CONFIGS["3"]
    p, V, W, A, bias, dM, dV0 = run_case(case, seed=12)
    # sums are formed in a fixed order: two runs agree bit for bit
    outs = []
    for _ in range(2):
        dV = dV0.clone()
        _, dW, dA = dma.dma_mask_bwd(p, V, W, A, bias, dM, dV)
        torch.cuda.synchronize()
        outs.append((dV.clone(), dW.clone(), dA.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_argument_checks():
    case = wl.small(wl.CONFIGS["2"], B=1, Hq=2, Hkv=1, L=128, d=128, w=32, name="mask-bwd-args")
    p = problem_of(case)
    dev = torch.device("cuda:0")
    V = torch.zeros(1, 128, 1, 128, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(2, 128, device=dev); A = torch.ones(2, device=dev)
    bias = torch.ones(1, 2, 128, device=dev); dM = torch.zeros(1, 2, 128, device=dev)
    tiny = torch.empty(16, dtype=torch.uint8, device=dev)
    with pytest.raises(dma.DmaError) as e:
        dma.dma_mask_bwd(p, V, W, A, bias, dM, V.clone(), ws=tiny)
    assert e.value.status == -5
