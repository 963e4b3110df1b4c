"""dma_mask_build_static: the mask build for hosts that may not allocate device memory when the mask is built
(an arena-owning server, a plug-in without an allocator). Its scratch is a fixed array inside the library, so the
check is simply that it gives the same bits as dma_mask_build, call after call, and refuses what does not fit.
Collected last on purpose (file name), so that a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def build_both(case, inp, out, causal=1, full=False):
    dev = torch.device("cuda:0")
    p = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, causal=causal,
                    flags=dma.DMA_FLAG_FULL_DELTA if full else 0)
    V, A = inp["V"].to(dev), inp["A"].to(dev)
    W = (wl.full_delta_weights(case) if full else inp["W_delta"]).to(dev)
    ref = dma.dma_mask_build(p, V, W, A)
    for t in out:
        t.fill_(-1)                                   # outputs are preallocated by the caller and fully overwritten
    dma.dma_mask_build_static(p, V, W, A, *out)
    torch.cuda.synchronize()
    for name, a, b in zip(("bias", "expiry", "bitmap"), ref, out):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), name     # bit-exact, as for every mask test


def test_static_scratch_matches_workspace_version_on_consecutive_calls():
    dev = torch.device("cuda:0")
    # two different problems back to back: the second call finds the first call's contents in the shared array
    big = wl.small(wl.CONFIGS["2"], B=1, Hq=8, Hkv=2, L=3000, w=500, name="static-a")
    small = wl.small(wl.CONFIGS["1"], B=2, Hq=2, Hkv=2, L=300, w=37, name="static-b")
    for case in (big, small, big):
        out = (torch.empty(case.B, case.Hq, case.L, dtype=torch.float32, device=dev),
               torch.empty(case.B, case.Hq, case.L, dtype=torch.int32, device=dev),
               torch.empty(case.B, case.Hq, -(-case.L // 128), (-(-case.L // 128) + 31) // 32, dtype=torch.int32, device=dev))
        inp = wl.make_inputs(case)
        build_both(case, inp, out)
        build_both(case, inp, out)
        build_both(case, inp, out, causal=0)                      # the non-causal selection and the full sampling weights
        build_both(case, inp, out, full=True)                     # go through the same scratch


@pytest.mark.parametrize("Hq,Hkv,L", [(32, 8, 32768), (1, 1, 1 << 20)])
def test_static_scratch_at_exactly_its_limit(Hq, Hkv, L):
    # 1,048,576 sort keys in all, as 32 heads of 32768 keys or as one head of 2^20 keys: the one head needs all 20 levels of
    # the rank tree the array has room for, so its last level ends on the array's last byte. V is the recipe's noise; the
    # check is bit-equality with the workspace version, twice in a row.
    dev = torch.device("cuda:0")
    case = wl.small(wl.CONFIGS["3"], B=1, Hq=Hq, Hkv=Hkv, L=L, d=64, w=1000, name="static-limit")
    g = torch.Generator().manual_seed(77)
    inp = {"V": torch.randn(case.B, case.L, case.Hkv, case.d, generator=g).to(case.torch_dtype),
           "W_delta": torch.randn(case.Hq, case.d, generator=g) / 8.0, "A": torch.rand(case.Hq, generator=g) * 1.5 + 0.5}
    T = case.L // 128
    out = (torch.empty(case.B, case.Hq, case.L, dtype=torch.float32, device=dev),
           torch.empty(case.B, case.Hq, case.L, dtype=torch.int32, device=dev),
           torch.empty(case.B, case.Hq, T, (T + 31) // 32, dtype=torch.int32, device=dev))
    build_both(case, inp, out)
    build_both(case, inp, out)
    one_more = dma.problem(case.B, case.Hq, case.Hkv, case.L + 1, case.d, case.w)      # one key over: a whole new chunk per head
    with pytest.raises(dma.DmaError) as e:
        dma.dma_mask_build_static(one_more, inp["V"].to(dev), inp["W_delta"].to(dev), inp["A"].to(dev), *out)
    assert e.value.status == -5


def test_static_scratch_rejects_oversized_problems():
    dev = torch.device("cuda:0")
    p = dma.problem(1, 32, 8, 65536, 128, 4096)      # 2 Mi sort keys: over the 1 Mi limit
    a = torch.empty(64, dtype=torch.float32, device=dev)
    v = torch.empty(64, dtype=torch.bfloat16, device=dev)     # refused before anything is read
    with pytest.raises(dma.DmaError) as e:
        dma.dma_mask_build_static(p, v, a, a, a, a.view(torch.int32), a.view(torch.int32))
    assert e.value.status == -5
