"""Randomised parity. The mask build against the oracle, bit for bit: random sizes (including L below one chunk and
ragged tails), window sizes around and above L, element types, head groupings, the three selection modes (causal, packed
documents, non-causal) and both sampling-weight shapes. The mask backward against the oracle, and forward chunks at random
positions against the whole forward."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("seed", range(24))
def test_mask_build_matches_the_oracle(seed):
    r = np.random.default_rng(500 + seed)
    Hkv = int(r.choice([1, 2, 3, 4]))
    G = int(r.choice([1, 2, 4]))
    L = int(r.choice([1, 7, 255, 256, 257, 700, 1500, 2900]))
    w = int(r.choice([1, 2, 33, 256, 1000, L, L + 50]))
    d = int(r.choice([64, 128]))
    dtype = str(r.choice(["bf16", "fp32"]))
    mode = str(r.choice(["causal", "varlen", "noncausal"]))
    full = bool(r.integers(0, 2))
    case = wl.small(wl.CONFIGS["2"], B=int(r.choice([1, 2])), Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, dtype=dtype, seed=3000 + seed,
                    boost_rows=int(r.choice([0, 5])) if L > 16 else 0, name=f"mask-stress-{seed}")
    inp = wl.make_inputs(case)
    if seed % 5 == 0:
        inp["A"][0] = 0.0                                          # one head with every delta equal: ties by index
    W = wl.full_delta_weights(case) if full else inp["W_delta"]
    Vf = inp["V"].float().numpy()
    dl = oracle.delta_full(Vf, W.numpy(), inp["A"].numpy())[1] if full else oracle.delta(Vf, W.numpy(), inp["A"].numpy(), case.Hq)[1]
    p = dma.problem(case.B, case.Hq, case.Hkv, L, d, w, dtype=case.torch_dtype, causal=0 if mode == "noncausal" else 1,
                    flags=dma.DMA_FLAG_FULL_DELTA if full else 0)
    V, Wd, A = inp["V"].to(DEV), W.to(DEV), inp["A"].to(DEV)
    if mode == "varlen":
        nseq = int(r.integers(1, min(L, 6) + 1))
        cu = [0] + sorted(set(int(c) for c in r.integers(1, max(L, 2), nseq - 1) if c < L)) + [L]
        got = dma.dma_mask_build_varlen(p, V, Wd, A, torch.tensor(cu, dtype=torch.int32, device=DEV))
        e = oracle.select_expiry_varlen(dl, min(w, L), cu)
        bmp = oracle.bitmap_from_expiry(e)
    elif mode == "noncausal":
        got = dma.dma_mask_build(p, V, Wd, A)
        e = oracle.select_noncausal(dl, w)
        bmp = oracle.bitmap_definition(oracle.keep_from_expiry_noncausal(e)) if L <= 1500 else None
    else:
        got = dma.dma_mask_build(p, V, Wd, A)
        e = oracle.select_expiry(dl, min(w, L))
        bmp = oracle.bitmap_from_expiry(e)
    torch.cuda.synchronize()
    info = (seed, mode, full, dtype, case.B, case.Hq, Hkv, L, w, d)
    assert np.array_equal(got[0].cpu().numpy().view(np.uint32), dl.view(np.uint32)), info
    assert np.array_equal(got[1].cpu().numpy(), e), info
    if bmp is not None:
        assert np.array_equal(got[2].cpu().numpy().view(np.uint32), bmp), info


@pytest.mark.parametrize("seed", range(12))
def test_mask_backward_matches_the_oracle(seed):
    from helpers import assert_close
    r = np.random.default_rng(700 + seed)
    Hkv = int(r.choice([1, 2, 3]))
    G = int(r.choice([1, 2, 4, 8]))
    L = int(r.choice([1, 63, 64, 65, 500, 1300]))
    d = int(r.choice([64, 128]))
    dtype = str(r.choice(["bf16", "fp32"]))
    full = bool(r.integers(0, 2))
    case = wl.small(wl.CONFIGS["2"], B=int(r.choice([1, 3])), Hq=Hkv * G, Hkv=Hkv, L=L, w=max(1, L // 3), d=d, dtype=dtype,
                    seed=4000 + seed, name=f"mask-bwd-stress-{seed}")
    inp = wl.make_inputs(case)
    W = wl.full_delta_weights(case) if full else inp["W_delta"]
    p = dma.problem(case.B, case.Hq, case.Hkv, L, d, case.w, dtype=case.torch_dtype, flags=dma.DMA_FLAG_FULL_DELTA if full else 0)
    V, Wd, A = inp["V"].to(DEV), W.to(DEV), inp["A"].to(DEV)
    bias, _, _ = dma.dma_mask_build(p, V, Wd, A)
    g = torch.Generator().manual_seed(seed)
    dM = torch.randn(case.B, case.Hq, L, generator=g)
    dV0 = torch.randn(case.B, L, Hkv, d, generator=g).to(case.torch_dtype)
    dV = dV0.to(DEV).clone()
    _, dW, dA = dma.dma_mask_bwd(p, V, Wd, A, bias, dM.to(DEV), dV)
    torch.cuda.synchronize()
    if full:
        rV, rW, rA = oracle.mask_backward_full(inp["V"].double().numpy(), W.double().numpy(), inp["A"].double().numpy(), dM.double().numpy())
    else:
        rV, rW, rA = oracle.mask_backward(inp["V"].double().numpy(), W.double().numpy(), inp["A"].double().numpy(), dM.double().numpy(), case.Hq)
    info = f"seed {seed} full {full} {dtype} B{case.B} Hq{case.Hq} Hkv{Hkv} L{L} d{d}"
    assert_close(dV, dV0.double().numpy() + rV, dtype, info + ": dV")
    assert_close(dW, rW, "fp32", info + ": dW")
    assert_close(dA, rA, "fp32", info + ": dA")


@pytest.mark.parametrize("seed", range(10))
def test_forward_chunks_match_the_whole_forward(seed):
    r = np.random.default_rng(900 + seed)
    Hkv, G = int(r.choice([1, 2])), int(r.choice([1, 2, 4]))
    L = int(r.choice([300, 777, 1024, 2500]))
    d = int(r.choice([64, 128]))
    case = wl.small(wl.CONFIGS["2"], B=int(r.choice([1, 2])), Hq=Hkv * G, Hkv=Hkv, L=L, w=int(r.choice([1, 40, 300])), d=d,
                    seed=5000 + seed, name=f"chunk-stress-{seed}")
    inp = wl.make_inputs(case)
    p = dma.problem(case.B, case.Hq, case.Hkv, L, d, case.w)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(DEV), inp["A"].to(DEV))
    ps = dma.problem(case.B, case.Hq, case.Hkv, L, d, case.w, flags=dma.DMA_FLAG_SIMT)
    ref, lref = dma.dma_attn_fwd(ps, Q, K, V, bias, expiry, bitmap)
    for _ in range(4):
        q_begin = int(r.integers(0, L))
        q_len = int(r.integers(1, L - q_begin + 1))
        O, lse = dma.dma_attn_fwd_chunk(p, q_begin, Q[:, q_begin:q_begin + q_len].contiguous(), K, V, bias, expiry)
        torch.cuda.synchronize()
        assert float((O.float() - ref[:, q_begin:q_begin + q_len].float()).abs().max()) <= 3e-2, (seed, q_begin, q_len)
        assert float((lse - lref[:, :, q_begin:q_begin + q_len]).abs().max()) <= 1e-3 * max(1.0, float(lref.abs().max())), (seed, q_begin, q_len)
