"""GPU parity for sequences packed along the sequence axis (dma_mask_build_varlen): the mask bit for bit against the
oracle's per-sequence selection, and the unchanged attention kernels on the resulting block-diagonal masks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close, f64, problem_of, round_to, stored_forward
from test_gpu_attention import compare, oracle_all

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]

SMALL = [
    (wl.small(C1, L=37, w=4, name="varlen fp32 tiny"), [0, 5, 6, 20, 37]),
    (wl.small(C1, B=2, L=600, w=64, name="varlen fp32 boundaries inside a chunk"), [0, 100, 255, 256, 257, 511, 600]),
    (wl.small(C1, L=300, w=500, name="varlen fp32 w above every length"), [0, 140, 300]),
    (wl.small(C2, B=1, Hq=4, Hkv=2, L=1000, w=129, backward=True, name="varlen bf16 ragged gqa"), [0, 1, 333, 334, 900, 1000]),
    (wl.small(C2, B=2, Hq=4, Hkv=1, L=1536, w=200, backward=True, name="varlen bf16 three documents"), [0, 700, 829, 1536]),
    (wl.small(C2, B=1, Hq=2, Hkv=2, L=1024, w=64, backward=True, name="varlen bf16 tile-aligned"), [0, 256, 512, 1024]),
    (wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=64, backward=True, name="varlen bf16 d64"), [0, 77, 300, 512]),
    (wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=128, backward=True, name="varlen bf16 late entry"), [0, 77, 300, 512]),
    (wl.small(C2, B=1, Hq=2, Hkv=1, L=700, w=1, backward=True, name="varlen bf16 w=1"), [0, 130, 131, 400, 700]),
    (wl.small(C1, B=1, L=40, w=3, name="varlen fp32 every document one token"), list(range(41))),
]


def patched(case, O, lse, stored):
    """The GPU forward's O / lse with the oracle's stored values written over all rows or over the listed rows (the
    backward's inputs: Alg. 2 reads the stored forward output, and both backward passes are given the same one)."""
    if stored is None:
        return O, lse
    so, sl = torch.from_numpy(stored["O"]).to(case.torch_dtype).to(DEV), torch.from_numpy(stored["lse"]).to(DEV)
    if stored["rows"] is None:
        return so.contiguous(), sl.contiguous()
    idx = torch.from_numpy(stored["rows"].astype(np.int64)).to(DEV)
    O, lse = O.clone(), lse.clone()
    O[:, idx] = so
    lse[:, :, idx] = sl
    return O, lse


def run(case, cu, flags=0, backward=True, stored=None, inp=None):
    inp = wl.make_inputs(case) if inp is None else inp
    p = problem_of(case, flags=flags)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    cu_t = torch.tensor(cu, dtype=torch.int32, device=DEV)
    bias, expiry, bitmap = dma.dma_mask_build_varlen(p, V, inp["W_delta"].to(DEV), inp["A"].to(DEV), cu_t)
    O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
    got = {"bias": bias, "expiry": expiry, "bitmap": bitmap, "O": O, "lse": lse}
    if backward:
        O_in, lse_in = patched(case, O, lse, stored)
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O_in, dO, lse_in, bias, expiry, bitmap)
        got.update(dQ=dQ, dK=dK, dV=dV, dM=dM)
    torch.cuda.synchronize()
    return inp, got


def oracle_varlen_mask(case, inp, cu):
    _, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), inp["A"].numpy(), case.Hq)
    e = oracle.select_expiry_varlen(dl, min(case.w, case.L), cu)
    return dl, e, oracle.bitmap_from_expiry(e)


@pytest.mark.parametrize("case,cu", SMALL, ids=lambda v: v.name if hasattr(v, "name") else "")
def test_mask_and_attention_small(case, cu):
    inp = wl.make_inputs(case)
    dl, e, bmp = oracle_varlen_mask(case, inp, cu)
    ref = oracle_all(case, inp, dl, e)
    _, got = run(case, cu, stored=stored_forward(case, ref["O"], ref["lse"]), inp=inp)
    assert np.array_equal(got["bias"].cpu().numpy().view(np.uint32), dl.view(np.uint32))
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    assert np.array_equal(got["bitmap"].cpu().numpy().view(np.uint32), bmp)
    compare(case, got, ref)


@pytest.mark.parametrize("case,cu", [c for c in SMALL if c[0].dtype == "bf16" and c[0].d == 128],
                         ids=lambda v: v.name if hasattr(v, "name") else "")
def test_token_compacted_kernels_on_packed_sequences(case, cu):
    inp = wl.make_inputs(case)
    dl, e, _ = oracle_varlen_mask(case, inp, cu)
    ref = oracle_all(case, inp, dl, e)
    _, got = run(case, cu, flags=dma.DMA_FLAG_COMPACT_KV, stored=stored_forward(case, ref["O"], ref["lse"]), inp=inp)
    compare(case, got, ref)


def test_query_tile_whose_first_key_tiles_belong_to_another_document():
    """Regression: the second query tile of a CTA's pair starts a new document, so it skips the key tiles its partner
    still needs and enters the walk late, at a tile that takes the per-element path. It once read that tile's fast-path
    flag before the stager had written it (the outcome depended on where the tensors lay in memory). Several placements
    of Q, K, V, tensor-core kernel against the CUDA-core kernel."""
    case = wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=128, backward=False, name="varlen late entry")
    cu = torch.tensor([0, 77, 300, 512], dtype=torch.int32, device=DEV)
    inp = wl.make_inputs(case)
    p, ps = problem_of(case), problem_of(case, flags=dma.DMA_FLAG_SIMT)
    n = case.L * case.Hq * case.d
    big = torch.empty(3 * n + (4 << 20), dtype=torch.bfloat16, device=DEV)
    W, A = inp["W_delta"].to(DEV), inp["A"].to(DEV)
    for trial in range(12):
        off = trial * 0x12340 * 4
        Q, K, V = (big[off + t * n:off + (t + 1) * n].view(1, case.L, case.Hq, case.d) for t in range(3))
        Q.copy_(inp["Q"]); K.copy_(inp["K"]); V.copy_(inp["V"])
        bias, expiry, bitmap = dma.dma_mask_build_varlen(p, V, W, A, cu)
        ref, lref = dma.dma_attn_fwd(ps, Q, K, V, bias, expiry, bitmap)
        O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
        torch.cuda.synchronize()
        assert float((O.float() - ref.float()).abs().max()) <= 3e-2, trial
        assert float((lse - lref).abs().max()) <= 1e-3 * max(1.0, float(lref.abs().max())), trial


def test_one_sequence_equals_the_plain_mask_build():
    case = wl.small(C2, B=1, Hq=4, Hkv=2, L=2000, w=300, name="varlen one sequence")
    inp = wl.make_inputs(case)
    p = problem_of(case)
    V, W, A = inp["V"].to(DEV), inp["W_delta"].to(DEV), inp["A"].to(DEV)
    a = dma.dma_mask_build(p, V, W, A)
    b = dma.dma_mask_build_varlen(p, V, W, A, torch.tensor([0, case.L], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_config3_packed_documents():
    """Config 3's shapes with 12 packed documents: expiry and bitmap bit-exact at full size; O, lse, dK, dV, dM on sampled
    rows and keys; no key tile of another document is ever active."""
    case = wl.CONFIGS["3"]
    cu = wl.packed_cu_seqlens(case.L, 12, seed=31)
    inp = wl.make_inputs(case)
    dl, e, bmp = oracle_varlen_mask(case, inp, cu)
    Q, K, V, dO = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
    rng = np.random.default_rng(5)
    L = case.L
    # sampled rows (document starts and ends included) and, for the gradients, every row of the last document: only its
    # rows can keep its keys. The oracle's forward on those rows is the stored O / lse that both backward passes read.
    s0 = cu[-2]
    rows = np.unique(np.concatenate([[0, L - 1], np.asarray(cu[1:-1]) - 1, np.asarray(cu[1:-1]), rng.integers(0, L, 12),
                                     np.arange(s0, L)])).astype(np.int32)
    O, lse = oracle.forward(Q, K, V, dl.astype(np.float64), expiry=e, rows=rows)
    st = stored_forward(case, O, lse, rows=rows)
    keys = np.unique(np.concatenate([[s0, L - 1], rng.integers(s0, L, 5)])).astype(np.int32)
    Ostored = np.zeros_like(Q)
    Ostored[:, rows] = st["O"]
    _, dK, dV, dM = oracle.backward(Q, K, V, dO, dl.astype(np.float64), expiry=e, keys=keys, want_dq=False, O=Ostored)
    dq = np.unique(np.concatenate([[s0, s0 + 1, L - 1], rng.integers(s0, L, 5)])).astype(np.int32)
    dQ = oracle.backward_dq_rows(Q, K, V, dO, dl.astype(np.float64), dq, expiry=e, O=st["O"][:, np.searchsorted(rows, dq)])

    _, got = run(case, cu, flags=dma.DMA_FLAG_TILE_PATH, stored=st, inp=inp)
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    assert np.array_equal(got["bitmap"].cpu().numpy().view(np.uint32), bmp)
    seq_of = np.searchsorted(np.asarray(cu), np.arange(case.L), side="right") - 1
    words = got["bitmap"].cpu().numpy().view(np.uint32)
    Tr = words.shape[2]
    for qt in range(Tr):
        first_seq_start = cu[seq_of[qt * 128]]
        for kt in range(first_seq_start // 128):                 # tiles wholly before the first document of the query tile
            assert not (words[:, :, qt, kt // 32] >> np.uint32(kt % 32) & np.uint32(1)).any()
    # the tile-walking kernels, then the token-compacted kernels on the same packed batch, against the same oracle samples
    for tag, g in (("", got), ("compact ", run(case, cu, flags=dma.DMA_FLAG_COMPACT_KV, stored=st, inp=inp)[1])):
        assert_close(g["O"][:, rows], O, case.dtype, tag + "O rows")
        assert_close(g["lse"][:, :, rows], lse, case.dtype, tag + "lse rows", lse=True)
        assert_close(g["dK"][:, keys], dK, case.dtype, tag + "dK keys")
        assert_close(g["dV"][:, keys], dV, case.dtype, tag + "dV keys")
        assert_close(g["dM"][:, :, keys], dM, case.dtype, tag + "dM keys")
        assert_close(g["dQ"][:, dq], dQ, case.dtype, tag + "dQ rows")


def test_argument_checks():
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=128, d=128, w=32, name="varlen args")
    p = problem_of(case)
    inp = wl.make_inputs(case)
    V, W, A = inp["V"].to(DEV), inp["W_delta"].to(DEV), inp["A"].to(DEV)
    with pytest.raises(dma.DmaError) as err:
        dma.dma_mask_build_varlen(p, V, W, A, torch.zeros(1, dtype=torch.int32, device=DEV))     # nseq = 0
    assert err.value.status == -2
