"""GPU parity of the non-causal mode (causal = 0: every row of a head keeps the same top-w keys): mask bit for bit,
forward and backward within the gate, on the CUDA-core kernels and on the token-compacted tensor-core kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, f64, round_to, stored_forward
from test_gpu_varlen import patched

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]

CASES = [
    wl.small(C1, L=256, w=64, name="nc fp32"),
    wl.small(C1, L=1, w=1, name="nc fp32 L1"),
    wl.small(C1, L=77, w=200, name="nc fp32 w>=L ragged"),
    wl.small(C1, B=2, d=128, Hq=4, Hkv=2, L=321, w=50, name="nc fp32 d128 gqa ragged"),
    wl.small(C2, B=2, Hq=4, Hkv=2, L=1000, w=129, backward=True, name="nc bf16 ragged gqa"),
    wl.small(C2, B=1, Hq=8, Hkv=2, L=1024, w=256, backward=True, name="nc bf16 L1024"),
    wl.small(C2, B=1, Hq=2, Hkv=1, L=640, w=1, backward=True, name="nc bf16 w=1"),
    wl.small(C2, B=1, Hq=2, Hkv=2, L=130, w=999, backward=True, name="nc bf16 dense"),
    wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=64, backward=True, name="nc bf16 d64"),
    wl.small(C2, B=1, Hq=4, Hkv=1, L=1536, w=200, backward=True, qk_scale=3.0, name="nc bf16 peaked"),
]


def inputs(case):
    """The case's seeded inputs with the gate A scaled by 1/4. Every row of a head shares one key set here, and with the
    causal recipe's gates (delta up to several hundred) the best key's bias outweighs all others in EVERY row: the softmax
    is one-hot, the exact dQ, dK, dM are ~1e-15 and a relative error against them measures nothing. With A/4 the biases
    stay within a few units of each other and all gradients are of ordinary size."""
    inp = wl.make_inputs(case)
    inp["A"] = inp["A"] * 0.25
    return inp


def problem(case, flags=0):
    return dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, causal=0, flags=flags)


def gpu(case, inp, flags=0, backward=True, stored=None):
    p = problem(case, flags)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(DEV), inp["A"].to(DEV))
    O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
    out = {"bias": bias, "expiry": expiry, "bitmap": bitmap, "O": O, "lse": lse}
    if backward:
        O_in, lse_in = patched(case, O, lse, stored)          # Alg. 2's stored forward output: the oracle's, for both sides
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O_in, dO, lse_in, bias, expiry, bitmap)
        out.update(dQ=dQ, dK=dK, dV=dV, dM=dM)
    torch.cuda.synchronize()
    return out


def oracle_mask(case, inp):
    _, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), inp["A"].numpy(), case.Hq)
    return dl, oracle.select_noncausal(dl, case.w)


def oracle_all(case, inp, dl, e):
    Q, K, V, dO = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
    O, lse = oracle.forward(Q, K, V, dl.astype(np.float64), expiry=e, causal=False)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, dl.astype(np.float64), expiry=e, O=round_to(case, O), causal=False)
    return {"O": O, "lse": lse, "dQ": dQ, "dK": dK, "dV": dV, "dM": dM}


def check_all(case, got, ref):
    assert_close(got["O"], ref["O"], case.dtype, "O")
    assert_close(got["lse"], ref["lse"], case.dtype, "lse", lse=True)
    for k in ("dQ", "dK", "dV", "dM"):
        assert_close(got[k], ref[k], case.dtype, k)


@pytest.mark.parametrize("case", CASES, ids=lambda c: c.name)
def test_mask_forward_backward_small(case):
    inp = inputs(case)
    dl, e = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    got = gpu(case, inp, stored=stored_forward(case, ref["O"], ref["lse"]))
    assert np.array_equal(got["bias"].cpu().numpy().view(np.uint32), dl.view(np.uint32))
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    keep = oracle.keep_from_expiry_noncausal(e)
    assert np.array_equal(got["bitmap"].cpu().numpy().view(np.uint32), oracle.bitmap_definition(keep))
    check_all(case, got, ref)


@pytest.mark.parametrize("case", [c for c in CASES if c.dtype == "bf16"], ids=lambda c: c.name)
def test_cuda_core_kernels_on_bf16(case):
    inp = inputs(case)
    dl, e = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    check_all(case, gpu(case, inp, flags=dma.DMA_FLAG_SIMT, stored=stored_forward(case, ref["O"], ref["lse"])), ref)


def test_last_row_equals_the_causal_last_row_on_the_gpu():
    case = wl.small(C2, B=1, Hq=4, Hkv=2, L=2048, w=300, name="nc last row")
    inp = inputs(case)
    got = gpu(case, inp, backward=False)
    pc = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype)
    Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
    bias, expiry, bitmap = dma.dma_mask_build(pc, V, inp["W_delta"].to(DEV), inp["A"].to(DEV))
    O, lse = dma.dma_attn_fwd(pc, Q, K, V, bias, expiry, bitmap)
    torch.cuda.synchronize()
    assert torch.equal(bias, got["bias"])
    assert (O[:, -1].float() - got["O"][:, -1].float()).abs().max() <= 2e-2
    assert (lse[..., -1] - got["lse"][..., -1]).abs().max() <= 1e-3 * max(1.0, float(lse[..., -1].abs().max()))


def test_config3_sampled():
    """Config 3's shapes: expiry bit-exact at full size; O, lse on sampled rows; dK, dV, dM on sampled kept and dropped keys
    of the first KV group (the oracle needs every row for a kept key, so the problem is cut to one group)."""
    case = wl.CONFIGS["3"]
    inp = inputs(case)
    dl, e = oracle_mask(case, inp)
    Q, K, V, dO = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
    G = case.Hq // case.Hkv
    # the first KV group in full on the oracle: its forward output is the stored O / lse that both backward passes read
    # for those heads (the other heads' backward, which is not compared, reads the GPU's own forward output)
    Og, lg = oracle.forward(Q[:, :, :G], K[:, :, :1], V[:, :, :1], dl[:, :G].astype(np.float64), expiry=e[:, :G], causal=False)
    p = problem(case)
    Qd, Kd, Vd, dOd = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    bias, expiry, bitmap = dma.dma_mask_build(p, Vd, inp["W_delta"].to(DEV), inp["A"].to(DEV))
    Od, lsed = dma.dma_attn_fwd(p, Qd, Kd, Vd, bias, expiry, bitmap)
    O_in, lse_in = Od.clone(), lsed.clone()
    O_in[:, :, :G] = torch.from_numpy(round_to(case, Og)).to(case.torch_dtype).to(DEV)
    lse_in[:, :G] = torch.from_numpy(lg.astype(np.float32)).to(DEV)
    dQd, dKd, dVd, dMd = dma.dma_attn_bwd(p, Qd, Kd, Vd, O_in, dOd, lse_in, bias, expiry, bitmap)
    torch.cuda.synchronize()
    got = {"expiry": expiry, "O": Od, "lse": lsed, "dQ": dQd, "dK": dKd, "dV": dVd, "dM": dMd}
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    rng = np.random.default_rng(9)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, case.L - 1], rng.integers(0, case.L, 16)])).astype(np.int32)
    O, lse = oracle.forward(Q, K, V, dl.astype(np.float64), expiry=e, rows=rows, causal=False)
    assert_close(got["O"][:, rows], O, case.dtype, "O rows")
    assert_close(got["lse"][:, :, rows], lse, case.dtype, "lse rows", lse=True)
    kept = np.nonzero(e[0, :G].max(0))[0]
    dropped = np.nonzero(e[0, :G].max(0) == 0)[0]
    keys = np.unique(np.concatenate([rng.choice(kept, 4), rng.choice(dropped, 2)])).astype(np.int32)
    Qg, dOg = Q[:, :, :G], dO[:, :, :G]
    _, dK, dV, dM = oracle.backward(Qg, K[:, :, :1], V[:, :, :1], dOg, dl[:, :G].astype(np.float64), expiry=e[:, :G], keys=keys,
                                    want_dq=False, O=round_to(case, Og), causal=False)
    assert_close(got["dK"][:, keys, :1], dK, case.dtype, "dK keys")
    assert_close(got["dV"][:, keys, :1], dV, case.dtype, "dV keys")
    assert_close(got["dM"][:, :G, keys], dM, case.dtype, "dM keys")
    assert float(got["dM"][0, 0, torch.as_tensor(np.nonzero(e[0, 0] == 0)[0], device=DEV)].abs().max()) == 0.0


def test_varlen_needs_the_causal_mode():
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=128, d=128, w=32, name="nc varlen")
    inp = inputs(case)
    with pytest.raises(dma.DmaError) as err:
        dma.dma_mask_build_varlen(problem(case), inp["V"].to(DEV), inp["W_delta"].to(DEV), inp["A"].to(DEV),
                                  torch.tensor([0, 128], dtype=torch.int32, device=DEV))
    assert err.value.status == -4
