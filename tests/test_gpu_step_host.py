"""dma_step_host (the whole path on host buffers, cut into independent (batch, KV-head group) problems and pipelined with
the copies) against the device entry points on the same inputs, and against the oracle on a small case."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, gpu_run, oracle_mask, problem_of
from test_gpu_attention import compare, oracle_all

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]


def host_step(case, inp, flags=0, W=None):
    p = problem_of(case, flags=flags)
    W = inp["W_delta"] if W is None else W
    arena = torch.empty(dma.dma_step_host_arena(p, case.backward), dtype=torch.uint8, device=DEV)
    hO = torch.empty_like(inp["Q"]); hlse = torch.empty(case.B, case.Hq, case.L)
    hdQ, hdK, hdV = torch.full_like(inp["Q"], 7.0), torch.full_like(inp["K"], 7.0), torch.full_like(inp["V"], 7.0)
    hdM = torch.full((case.B, case.Hq, case.L), 7.0)
    dma.dma_step_host(p, case.backward, inp["Q"], inp["K"], inp["V"], inp["dO"], W, inp["A"], hO, hlse, hdQ, hdK, hdV, hdM, arena)
    out = {"O": hO, "lse": hlse}
    if case.backward:
        out.update(dQ=hdQ, dK=hdK, dV=hdV, dM=hdM)
    return out


@pytest.mark.parametrize("case", [
    wl.small(C2, B=2, Hq=16, Hkv=8, L=1024, w=256, backward=True, name="host bf16 2 batches x 4 head groups"),
    wl.small(C2, B=1, Hq=8, Hkv=2, L=640, w=100, backward=True, name="host bf16 2 head groups"),
    wl.small(C2, B=3, Hq=4, Hkv=2, L=333, w=50, backward=True, name="host bf16 ragged: batch groups only"),
    wl.small(C2, B=2, Hq=8, Hkv=4, L=512, w=64, backward=False, name="host bf16 forward only"),
    wl.small(C1, B=2, Hq=8, Hkv=2, L=256, w=64, name="host fp32"),
    # Hq * L not a multiple of four: a batch entry's vectors would start off a 16-byte boundary inside [B, Hq, L] arrays
    wl.small(C2, B=3, Hq=1, Hkv=1, L=333, w=64, backward=True, name="host bf16 one head, odd length"),
    wl.small(C2, B=2, Hq=2, Hkv=2, L=1, w=64, d=64, backward=True, name="host bf16 single key"),
    wl.small(C2, B=70, Hq=2, Hkv=1, L=130, w=20, backward=True, name="host bf16 more batch entries than groups"),
], ids=lambda c: c.name)
def test_equals_the_device_entry_points(case):
    inp = wl.make_inputs(case)
    got = host_step(case, inp)
    dev = gpu_run(case, inp, backward=case.backward)
    assert torch.equal(got["O"], dev["O"].cpu()) and torch.equal(got["lse"], dev["lse"].cpu())
    if case.backward:
        # dK, dV, dM are formed in a fixed order per key tile; dQ is accumulated with atomics (order-dependent rounding)
        for k in ("dK", "dV"):
            assert torch.equal(got[k], dev[k].cpu()), k
        assert_close(got["dM"], dev["dM"].double().cpu().numpy(), case.dtype, "dM")
        assert_close(got["dQ"], dev["dQ"].double().cpu().numpy(), case.dtype, "dQ")


def test_against_the_oracle():
    case = wl.small(C2, B=2, Hq=8, Hkv=4, L=512, w=96, backward=True, name="host oracle")
    inp = wl.make_inputs(case)
    got = host_step(case, inp)
    dl, e, _ = oracle_mask(case, inp)
    compare(case, got, oracle_all(case, inp, dl, e), end_to_end=True)


def test_flags_that_keep_the_batch_entries_whole():
    case = wl.small(C2, B=2, Hq=8, Hkv=4, L=512, w=96, backward=True, name="host flags")
    inp = wl.make_inputs(case)
    dl, e, _ = oracle_mask(case, inp)
    compare(case, host_step(case, inp, flags=dma.DMA_FLAG_COMPACT_KV), oracle_all(case, inp, dl, e), end_to_end=True)
    W = wl.full_delta_weights(case)
    _, dlf = oracle.delta_full(inp["V"].float().numpy(), W.numpy(), inp["A"].numpy())
    ef = oracle.select_expiry(dlf, case.w)
    compare(case, host_step(case, inp, flags=dma.DMA_FLAG_FULL_DELTA, W=W), oracle_all(case, inp, dlf, ef), end_to_end=True)
