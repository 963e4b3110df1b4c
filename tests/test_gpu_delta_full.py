"""GPU parity of the full sampling-weight projection (Eq. delta_calc with W over all Hkv*d value channels, flag
DMA_FLAG_FULL_DELTA): mask generation bit for bit, its backward within the floating-point gate."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, problem_of

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FULL = dma.DMA_FLAG_FULL_DELTA

SMALL = [
    dict(B=1, Hq=2, Hkv=2, L=256, d=64, w=64, dtype="fp32"),
    dict(B=2, Hq=4, Hkv=2, L=300, d=64, w=64, dtype="bf16"),          # ragged tail, d = 64
    dict(B=2, Hq=6, Hkv=3, L=517, d=128, w=128, dtype="bf16"),        # three KV heads, ragged tail
    dict(B=1, Hq=4, Hkv=4, L=1024, d=128, w=256, dtype="fp32"),
    dict(B=1, Hq=9, Hkv=1, L=70, d=128, w=32, dtype="bf16"),          # head count not a multiple of 8
]


def build(case, W=None, flags=FULL):
    inp = wl.make_inputs(case)
    W = wl.full_delta_weights(case) if W is None else W
    p = problem_of(case, flags=flags)
    V, A = inp["V"].to(DEV), inp["A"].to(DEV)
    bias, expiry, bitmap = dma.dma_mask_build(p, V, W.to(DEV), A)
    torch.cuda.synchronize()
    return inp, W, p, V, A, bias, expiry, bitmap


@pytest.mark.parametrize("kw", SMALL)
def test_mask_build_bit_exact(kw):
    case = wl.small(wl.CONFIGS["2"], name="full-delta-small", **kw)
    inp, W, p, V, A, bias, expiry, bitmap = build(case)
    _, dl = oracle.delta_full(inp["V"].float().numpy(), W.numpy(), inp["A"].numpy())
    assert np.array_equal(bias.cpu().numpy().view(np.uint32), dl.view(np.uint32))
    e = oracle.select_expiry(dl, case.w)
    assert np.array_equal(expiry.cpu().numpy(), e)
    assert np.array_equal(bitmap.cpu().numpy(), oracle.bitmap_from_expiry(e))


def test_config3_bit_exact_and_delta_range_agrees():
    case = wl.CONFIGS["3"]
    inp, W, p, V, A, bias, expiry, _ = build(case)
    _, dl = oracle.delta_full(inp["V"].float().numpy(), W.numpy(), inp["A"].numpy())
    assert np.array_equal(bias.cpu().numpy().view(np.uint32), dl.view(np.uint32))
    assert np.array_equal(expiry.cpu().numpy(), oracle.select_expiry(dl, case.w))
    # the decoding cache's append path computes the same bits, over a range with a ragged start and end
    cache = torch.zeros(case.B, case.Hq, case.L + 40, device=DEV)
    dma.dma_delta_range(p, V, W.to(DEV), A, cache, 0, 1000)
    dma.dma_delta_range(p, V, W.to(DEV), A, cache, 1000, case.L - 3)
    torch.cuda.synchronize()
    assert torch.equal(cache[:, :, :case.L - 3], bias[:, :, :case.L - 3])
    assert float(cache[:, :, case.L - 3:].abs().max()) == 0.0


def test_block_diagonal_weights_reproduce_the_per_head_path():
    case = wl.small(wl.CONFIGS["3"], L=4096, name="full-delta-blockdiag")
    inp = wl.make_inputs(case)
    G, d = case.Hq // case.Hkv, case.d
    W = torch.zeros(case.Hq, case.Hkv * d)
    for h in range(case.Hq):
        W[h, (h // G) * d:(h // G + 1) * d] = inp["W_delta"][h]
    _, _, _, _, _, bias, expiry, bitmap = build(case, W=W)
    _, _, _, _, _, bias_h, expiry_h, bitmap_h = build(case, W=inp["W_delta"], flags=0)
    assert torch.equal(bias, bias_h) and torch.equal(expiry, expiry_h) and torch.equal(bitmap, bitmap_h)


def run_bwd(case, seed):
    inp, W, p, V, A, bias, _, _ = build(case)
    g = torch.Generator().manual_seed(seed)
    dM = torch.randn(case.B, case.Hq, case.L, generator=g)
    dV0 = torch.randn(case.B, case.L, case.Hkv, case.d, generator=g).to(case.torch_dtype)
    dV = dV0.to(DEV).clone()
    _, dW, dA = dma.dma_mask_bwd(p, V, W.to(DEV), A, bias, dM.to(DEV), dV)
    torch.cuda.synchronize()
    assert dW.shape == (case.Hq, case.Hkv * case.d)
    rV, rW, rA = oracle.mask_backward_full(inp["V"].double().numpy(), W.double().numpy(), inp["A"].double().numpy(),
                                           dM.double().numpy())
    assert_close(dV, dV0.double().numpy() + rV, case.dtype, f"{case.name}: dV (in/out)")
    assert_close(dW, rW, "fp32", f"{case.name}: dW_delta")
    assert_close(dA, rA, "fp32", f"{case.name}: dA")
    return p, V, W.to(DEV), A, bias, dM.to(DEV), dV0.to(DEV)


@pytest.mark.parametrize("kw", SMALL)
def test_mask_bwd_small(kw):
    run_bwd(wl.small(wl.CONFIGS["2"], name="full-delta-bwd-small", backward=True, **kw), seed=21)


def test_mask_bwd_config3_and_reproducible():
    p, V, W, A, bias, dM, dV0 = run_bwd(wl.CONFIGS["3"], seed=22)
    outs = []
    for _ in range(2):
        dV = dV0.clone()
        _, dW, dA = dma.dma_mask_bwd(p, V, W, A, bias, dM, dV)
        torch.cuda.synchronize()
        outs.append((dV.clone(), dW.clone(), dA.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_too_many_weights_for_shared_memory_is_refused():
    case = wl.small(wl.CONFIGS["2"], B=1, Hq=64, Hkv=8, L=128, d=128, w=32, name="full-delta-big")
    p = problem_of(case, flags=FULL)
    V = torch.zeros(1, 128, 8, 128, dtype=torch.bfloat16, device=DEV)
    W = torch.zeros(64, 1024, device=DEV); A = torch.ones(64, device=DEV)
    with pytest.raises(dma.DmaError) as e:
        dma.dma_mask_build(p, V, W, A)
    assert e.value.status == -4


def test_with_packed_documents_and_without_the_causal_mask():
    """The full projection only changes delta: the packed-document and the non-causal selections on top of it stay exact."""
    case = wl.small(wl.CONFIGS["2"], B=1, Hq=4, Hkv=2, L=900, d=128, w=100, name="full-delta modes")
    inp = wl.make_inputs(case)
    W = wl.full_delta_weights(case)
    _, dl = oracle.delta_full(inp["V"].float().numpy(), W.numpy(), inp["A"].numpy())
    V, A = inp["V"].to(DEV), inp["A"].to(DEV)
    cu = [0, 17, 300, 301, 900]
    p = problem_of(case, flags=FULL)
    bias, expiry, bitmap = dma.dma_mask_build_varlen(p, V, W.to(DEV), A, torch.tensor(cu, dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    e = oracle.select_expiry_varlen(dl, case.w, cu)
    assert np.array_equal(bias.cpu().numpy().view(np.uint32), dl.view(np.uint32))
    assert np.array_equal(expiry.cpu().numpy(), e)
    assert np.array_equal(bitmap.cpu().numpy().view(np.uint32), oracle.bitmap_from_expiry(e))
    pn = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, causal=0, flags=FULL)
    bias, expiry, _ = dma.dma_mask_build(pn, V, W.to(DEV), A)
    torch.cuda.synchronize()
    assert np.array_equal(bias.cpu().numpy().view(np.uint32), dl.view(np.uint32))
    assert np.array_equal(expiry.cpu().numpy(), oracle.select_noncausal(dl, case.w))
