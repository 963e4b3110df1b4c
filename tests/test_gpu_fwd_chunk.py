"""GPU parity of dma_attn_fwd_chunk (forward over a chunk of query rows against the whole key sequence: prefill in pieces)
against the oracle's forward on those rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, f64, gpu_mask, oracle_mask, problem_of

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]


def run_chunks(case, chunks):
    inp = wl.make_inputs(case)
    p, bias, expiry, _ = gpu_mask(case, inp)
    dl, e, _ = oracle_mask(case, inp)
    assert np.array_equal(expiry.cpu().numpy(), e)
    Q64, K64, V64 = (f64(inp[k]) for k in ("Q", "K", "V"))
    K, V = inp["K"].to(DEV), inp["V"].to(DEV)
    for q_begin, q_len in chunks:
        Qc = inp["Q"][:, q_begin:q_begin + q_len].contiguous().to(DEV)
        O, lse = dma.dma_attn_fwd_chunk(p, q_begin, Qc, K, V, bias, expiry)
        torch.cuda.synchronize()
        rows = np.arange(q_begin, q_begin + q_len, dtype=np.int32)
        Or, lr = oracle.forward(Q64, K64, V64, dl.astype(np.float64), expiry=e, rows=rows)
        assert O.shape == (case.B, q_len, case.Hq, case.d) and lse.shape == (case.B, case.Hq, q_len)
        assert_close(O, Or, case.dtype, f"{case.name}: O rows {q_begin}+{q_len}")
        assert_close(lse, lr, case.dtype, f"{case.name}: lse rows {q_begin}+{q_len}", lse=True)


@pytest.mark.parametrize("case", [
    wl.small(C2, B=2, Hq=4, Hkv=2, L=1000, w=129, name="chunk bf16 ragged gqa"),
    wl.small(C2, B=1, Hq=8, Hkv=2, L=2048, w=256, name="chunk bf16 L2048"),
    wl.small(C2, B=1, Hq=2, Hkv=2, L=130, w=999, name="chunk bf16 dense-causal"),
    wl.small(C1, B=2, d=128, Hq=4, Hkv=2, L=321, w=50, name="chunk fp32 d128"),
    wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=64, name="chunk bf16 d64"),
], ids=lambda c: c.name)
def test_chunks_match_the_oracle(case):
    L = case.L
    chunks = [(0, L), (L - 1, 1), (0, 1), (L // 2, L - L // 2), (77, min(100, L - 77)), (L - min(L, 300), min(L, 300))]
    if L >= 1024:
        chunks += [(256, 512), (384, 129)]
    run_chunks(case, chunks)


def test_strided_chunk_views_and_full_size_config3():
    """The last 2048 rows of config 3 (a chunk of a 16K prefill) taken as a strided view of the full Q, written into a
    strided view of a full O; sampled rows against the oracle, all rows against dma_attn_fwd on the whole sequence."""
    case = wl.CONFIGS["3"]
    inp = wl.make_inputs(case)
    p, bias, expiry, bitmap = gpu_mask(case, inp)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    O_full, lse_full = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
    q_begin, q_len = case.L - 2048 - 37, 2048
    pc = problem_of(case)
    for sdst in (pc.q_stride, pc.o_stride):
        sdst[0], sdst[1], sdst[2] = Q.stride(0), Q.stride(1), Q.stride(2)
    O_buf = torch.zeros_like(Q)
    O, lse = dma.dma_attn_fwd_chunk(pc, q_begin, Q[:, q_begin:q_begin + q_len], K, V, bias, expiry, O=O_buf[:, q_begin:q_begin + q_len])
    torch.cuda.synchronize()
    assert float(O_buf[:, :q_begin].abs().max()) == 0.0 and float(O_buf[:, q_begin + q_len:].abs().max()) == 0.0
    assert (O.float() - O_full[:, q_begin:q_begin + q_len].float()).abs().max() <= 2e-2
    assert (lse - lse_full[:, :, q_begin:q_begin + q_len]).abs().max() <= 1e-3 * max(1.0, float(lse_full.abs().max()))
    dl, e, _ = oracle_mask(case, inp)
    rows = np.array([q_begin, q_begin + 1, q_begin + 1000, q_begin + q_len - 1], np.int32)
    Or, lr = oracle.forward(f64(inp["Q"]), f64(inp["K"]), f64(inp["V"]), dl.astype(np.float64), expiry=e, rows=rows)
    assert_close(O[:, rows - q_begin], Or, case.dtype, "O rows")
    assert_close(lse[:, :, rows - q_begin], lr, case.dtype, "lse rows", lse=True)


def test_argument_checks():
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=256, w=32, name="chunk args")
    inp = wl.make_inputs(case)
    p, bias, expiry, _ = gpu_mask(case, inp)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    for q_begin, rows in ((-1, 10), (250, 10), (100, 200)):          # before the sequence, past its end (twice)
        with pytest.raises(dma.DmaError) as err:
            dma.dma_attn_fwd_chunk(p, q_begin, torch.zeros(1, rows, 2, 128, dtype=torch.bfloat16, device=DEV), K, V, bias, expiry)
        assert err.value.status == -2
