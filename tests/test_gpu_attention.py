"""GPU parity of the attention forward (Sec. 4.2) and backward (Sec. 4.3) against the CPU oracle (fp64
instantiation, fed the same rounded inputs), through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl

from helpers import assert_close, f64, gpu_run, oracle_mask, problem_of, round_to, stored_forward

pytestmark = pytest.mark.gpu

C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]
CASES = [
    C1,
    wl.small(C1, L=1, w=1, name="fp32 L1"),
    wl.small(C1, L=77, w=200, name="fp32 w>=L ragged"),
    wl.small(C1, B=2, d=128, Hq=4, Hkv=2, L=321, w=50, name="fp32 d128 gqa ragged"),
    wl.small(C2, B=2, Hq=4, Hkv=2, L=1000, w=129, backward=True, name="bf16 ragged gqa"),
    wl.small(C2, B=1, Hq=8, Hkv=2, L=1024, w=256, backward=True, name="bf16 L1024"),
    wl.small(C2, B=1, Hq=2, Hkv=1, L=640, w=1, backward=True, name="bf16 w=1"),
    wl.small(C2, B=1, Hq=2, Hkv=2, L=130, w=999, backward=True, name="bf16 dense-causal"),
    wl.small(C2, B=1, Hq=4, Hkv=4, L=512, w=64, d=64, backward=True, name="bf16 d64"),
    wl.small(C2, B=1, Hq=4, Hkv=1, L=1536, w=200, backward=True, qk_scale=3.0, name="bf16 peaked"),
    # d = 64: the backward alternates between two P / dS buffers; schedules of one, two, three and five 64-row steps per CTA
    wl.small(C2, B=1, Hq=1, Hkv=1, L=64, w=16, d=64, backward=True, name="bf16 d64 one step"),
    wl.small(C2, B=2, Hq=2, Hkv=2, L=100, w=30, d=64, backward=True, name="bf16 d64 two steps"),
    wl.small(C2, B=1, Hq=2, Hkv=1, L=129, w=500, d=64, backward=True, name="bf16 d64 gqa three steps"),
    wl.small(C2, B=1, Hq=6, Hkv=2, L=300, w=41, d=64, backward=True, name="bf16 d64 group of 3 ragged"),
]


def oracle_all(case, inp, bias, e, backward=True):
    Q, K, V, dO = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
    O, lse = oracle.forward(Q, K, V, bias.astype(np.float64), expiry=e)
    out = {"O": O, "lse": lse}
    if backward:
        # Alg. 2 reads the stored forward output: D uses O rounded to the element type
        dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias.astype(np.float64), expiry=e, O=round_to(case, O))
        out.update(dQ=dQ, dK=dK, dV=dV, dM=dM)
    return out


def compare(case, got, ref, backward=True, end_to_end=False):
    """end_to_end: the GPU backward read the GPU forward's own stored O (dma_step_host cannot be handed another), which
    differs from the oracle's stored O wherever the two forwards round an element to different neighbours; D = rowsum(dO o O)
    of Alg. 2 carries those one-ulp differences into every dS of the row, so the gradients are held to the bound relative
    to the tensor's largest magnitude there. Everywhere else both backward passes read the same stored O and the
    per-row / per-head bounds apply."""
    assert_close(got["O"], ref["O"], case.dtype, "O")
    assert_close(got["lse"], ref["lse"], case.dtype, "lse", lse=True)
    if backward:
        for k in ("dQ", "dK", "dV", "dM"):
            assert_close(got[k], ref[k], case.dtype, k, kind="tensor" if end_to_end else None)


@pytest.mark.parametrize("case", CASES, ids=lambda c: c.name)
def test_forward_backward_small(case):
    inp = wl.make_inputs(case)
    dl, e, bmp = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    st = stored_forward(case, ref["O"], ref["lse"])          # both backward passes read the same stored forward output
    got = gpu_run(case, inp, stored=st)
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    compare(case, got, ref)
    # block skipping is an optimisation only: ignoring the bitmap must give the same result
    again = gpu_run(case, inp, stored=st, flags=dma.DMA_FLAG_IGNORE_BITMAP)
    compare(case, again, ref)


@pytest.mark.parametrize("case", [c for c in CASES if c.dtype == "bf16"], ids=lambda c: c.name)
def test_cuda_core_kernels_on_bf16(case):
    inp = wl.make_inputs(case)
    dl, e, bmp = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    compare(case, gpu_run(case, inp, stored=stored_forward(case, ref["O"], ref["lse"]), flags=dma.DMA_FLAG_SIMT), ref)


def test_injected_mask_zero_bias_is_dense_causal_attention():
    # any self-consistent (bias, expiry, bitmap) is accepted: zero bias + everything kept = textbook causal attention
    case = wl.small(C2, B=1, Hq=4, Hkv=2, L=700, w=700, backward=True, name="inject")
    inp = wl.make_inputs(case)
    B, Hq, L = case.B, case.Hq, case.L
    bias = np.zeros((B, Hq, L), np.float32)
    e = np.full((B, Hq, L), L, np.int32)
    bmp = oracle.bitmap_from_expiry(e).view(np.int32)
    ref_all = oracle_all(case, inp, bias, e)
    got = gpu_run(case, inp, mask=(bias, e, bmp), stored=stored_forward(case, ref_all["O"], ref_all["lse"]))
    q, k, v = (inp[n].double().permute(0, 2, 1, 3) for n in ("Q", "K", "V"))
    G = Hq // case.Hkv
    ref = torch.nn.functional.scaled_dot_product_attention(q, k.repeat_interleave(G, 1), v.repeat_interleave(G, 1), is_causal=True)
    assert_close(got["O"], ref.permute(0, 2, 1, 3).numpy(), "bf16", "O vs SDPA")
    compare(case, got, ref_all)


def test_skipped_tiles_do_not_change_the_result_on_a_banded_mask():
    # structured workload at reduced length: many inactive tiles
    case = wl.small(wl.CONFIGS["S"], L=2048, w=256, Hq=6, Hkv=2, name="S-small")
    inp = wl.make_inputs(case)
    dl, e, bmp = oracle_mask(case, inp)
    T = case.L // 128
    t = np.arange(T)
    active = ((bmp[..., t // 32] >> (t % 32)) & 1).sum()
    assert active < 0.8 * case.B * case.Hq * T * (T + 1) / 2           # the mask really has holes
    ref = oracle_all(case, inp, dl, e)
    st = stored_forward(case, ref["O"], ref["lse"])
    compare(case, gpu_run(case, inp, stored=st, flags=dma.DMA_FLAG_TILE_PATH), ref)
    compare(case, gpu_run(case, inp, stored=st, flags=dma.DMA_FLAG_IGNORE_BITMAP), ref)


def dq_rows(case):
    """Sampled query rows for dQ: the dense-causal region (rows below w keep every visible key) AND the region where
    the mask drops keys (rows at and beyond w), including both sides of a tile boundary and the last row."""
    L, w = case.L, min(case.w, case.L)
    rows = [0, 5, 130, min(700, L - 1), w - 1, min(w, L - 1), min(w + 1, L - 1), L // 2, (L // 2) | 1, 3 * L // 4 + 77,
            L - 129, L - 128, L - 1]
    return np.unique(np.clip(np.array(rows, np.int64), 0, L - 1)).astype(np.int32)


class Samples:
    """Full-size parity on sampled outputs: query rows (O, lse, dQ) and keys (dK, dV, dM) that the oracle evaluates one
    by one, computed BEFORE the GPU runs. Keys are sampled near the end of the sequence, where only the last 600 rows can
    keep them; dQ rows cover the region where the mask drops keys. `stored` holds the oracle's forward output on every
    row the sampled gradients depend on: the GPU backward is given those rows as its stored O / lse (Alg. 2 takes them
    as inputs), so both backward passes work from the same values."""

    def __init__(self, case, inp, nrows=24, nkeys=6, seed=0, forward_only=False):
        rng = np.random.default_rng(seed)
        self.case, self.inp = case, inp
        self.backward = case.backward and not forward_only
        self.dl, self.e, _ = oracle_mask(case, inp)
        Q, K, V, dO = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
        L, bias = case.L, self.dl.astype(np.float64)
        rows = np.concatenate([[0, 1, 127, 128, L - 1], rng.integers(0, L, nrows)])
        if self.backward:
            self.keys = np.unique(np.concatenate([[L - 1, L - 130], rng.integers(L - 600, L, nkeys)])).astype(np.int32)
            tail = np.arange(L - 600, L)                             # the only rows that can keep those keys
            self.dq = dq_rows(case)
            rows = np.concatenate([rows, tail, self.dq])
        self.rows = np.unique(rows).astype(np.int32)
        self.O, self.lse = oracle.forward(Q, K, V, bias, expiry=self.e, rows=self.rows)
        self.stored = stored_forward(case, self.O, self.lse, rows=self.rows)
        if self.backward:
            Ostored = np.zeros_like(Q)
            Ostored[:, self.rows] = self.stored["O"]                 # Alg. 2 reads the stored (rounded) forward output
            _, self.dK, self.dV, self.dM = oracle.backward(Q, K, V, dO, bias, expiry=self.e, keys=self.keys, want_dq=False, O=Ostored)
            at = np.searchsorted(self.rows, self.dq)
            self.dQ = oracle.backward_dq_rows(Q, K, V, dO, bias, self.dq, expiry=self.e, O=self.stored["O"][:, at])

    def check(self, got, tag=""):
        case = self.case
        assert_close(got["O"][:, self.rows], self.O, case.dtype, tag + "O rows")
        assert_close(got["lse"][:, :, self.rows], self.lse, case.dtype, tag + "lse rows", lse=True)
        if not self.backward:
            return
        assert_close(got["dK"][:, self.keys], self.dK, case.dtype, tag + "dK keys")
        assert_close(got["dV"][:, self.keys], self.dV, case.dtype, tag + "dV keys")
        assert_close(got["dM"][:, :, self.keys], self.dM, case.dtype, tag + "dM keys")
        assert_close(got["dQ"][:, self.dq], self.dQ, case.dtype, tag + "dQ rows")
        # properties that hold at any size (Sec. 4.3): rows of dS sum to zero; q.dQ and k.dK balance per KV group
        # (D is formed from the stored, rounded O, so each row of dS sums to dO_i.(O_i - stored O_i), at most
        # half a bf16 ulp of every |dO_ic O_ic| term; in fp32 the bound is the accumulation error)
        Q, K, dO = (f64(self.inp[k]) for k in ("Q", "K", "dO"))
        L = case.L
        dMs = f64(got["dM"]).sum(-1)
        half_ulp = 2.0 ** -9 if case.dtype == "bf16" else 2.0 ** -20
        bound = half_ulp * (np.abs(dO) * np.abs(f64(got["O"]))).sum((1, 3)) + 1e-3
        assert (np.abs(dMs) <= bound).all(), (dMs, bound)
        G = case.Hq // case.Hkv
        lhs = (Q * f64(got["dQ"])).sum(-1).reshape(case.B, L, case.Hkv, G).sum((1, 3))
        rhs = (K * f64(got["dK"])).sum(-1).sum(1)
        assert np.abs(lhs - rhs).max() <= 2e-2 * max(1.0, np.abs(rhs).max())


@pytest.mark.parametrize("key", ["2", "3", "3x3", "4w256", "4w2048", "4w8192", "5", "S"])
def test_full_size_configs_sampled(key):
    case = wl.CONFIGS[key]
    inp = wl.make_inputs(case)
    ref = Samples(case, inp)
    # the tile-walking kernels (Alg. 1 / Alg. 2 with block skipping)
    ref.check(gpu_run(case, inp, backward=case.backward, stored=ref.stored, flags=dma.DMA_FLAG_TILE_PATH))


def test_default_flags_choose_the_path_from_the_descriptor():
    """Without DMA_FLAG_COMPACT_KV / DMA_FLAG_TILE_PATH the library picks token-compacted execution for causal bf16 problems
    with L >= 2048 and 4 w <= L and the tile-walking kernels otherwise: O and lse are the bits of the explicitly chosen path,
    the injected over-full mask is reported (DMA_ERR_MASK_OVERFLOW) instead of being truncated silently."""
    dev = torch.device("cuda:0")
    for key, chosen in (("4w2048", dma.DMA_FLAG_COMPACT_KV), ("4w4096", dma.DMA_FLAG_TILE_PATH)):
        case = wl.small(wl.CONFIGS[key], Hq=4, Hkv=4, name="auto " + key)
        inp = wl.make_inputs(case)
        a, b = gpu_run(case, inp, backward=False), gpu_run(case, inp, backward=False, flags=chosen)
        assert torch.equal(a["O"], b["O"]) and torch.equal(a["lse"], b["lse"]), key
        sizes = [dma.dma_query_workspace(problem_of(case, flags=f)) for f in (0, chosen)]
        assert sizes[0] == sizes[1], key
    # a mask that keeps every visible key, declared with w = 64: the gathered lists (w + 256 entries) overflow
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=2048, w=64, name="overfull")
    inp = wl.make_inputs(case)
    p = problem_of(case, flags=dma.DMA_FLAG_COMPACT_KV)
    e = torch.full((1, 2, case.L), case.L, dtype=torch.int32, device=dev)
    bias = torch.zeros(1, 2, case.L, dtype=torch.float32, device=dev)
    bmp = torch.from_numpy(oracle.bitmap_from_expiry(e.cpu().numpy()).view(np.int32)).to(dev)
    ws = torch.empty(dma.dma_query_workspace(p)[1], dtype=torch.uint8, device=dev)
    dma.dma_attn_fwd(p, inp["Q"].to(dev), inp["K"].to(dev), inp["V"].to(dev), bias, e, bmp, ws=ws)
    assert dma.dma_read_status(ws) == -8


def test_mma_block_skipping_does_not_change_the_result():
    """With DMA_FLAG_BLOCK_SKIP the P V product of an executed tile leaves out the 16-key MMA blocks in which no key can be
    kept by the query tile's rows. P is exactly zero there, so O and lse must be the bits of the run with every block
    multiplied, on masks that really have such blocks: a banded importance
    pattern, packed documents whose boundaries fall inside key tiles, and the gathered lists of the token-compacted kernels.
    The same outputs are held to the oracle in the tests above."""
    dev = torch.device("cuda:0")
    banded = wl.small(wl.CONFIGS["S"], L=4096, w=200, Hq=6, Hkv=2, backward=False, name="block-skip banded")
    packed = wl.small(C2, B=1, Hq=4, Hkv=2, L=3000, w=300, backward=False, name="block-skip packed")
    for case, cu in ((banded, None), (packed, [0, 70, 1000, 1111, 1900, 2500, 3000])):
        inp = wl.make_inputs(case)
        Q, K, V = (inp[k].to(dev) for k in ("Q", "K", "V"))
        p0 = problem_of(case, flags=dma.DMA_FLAG_TILE_PATH)
        if cu is None:
            mask = dma.dma_mask_build(p0, V, inp["W_delta"].to(dev), inp["A"].to(dev))
        else:
            mask = dma.dma_mask_build_varlen(p0, V, inp["W_delta"].to(dev), inp["A"].to(dev), torch.tensor(cu, dtype=torch.int32, device=dev))
        # the mask must contain dead 16-key blocks inside active tiles, or the test checks nothing
        e = mask[1].cpu().numpy()
        bmp = mask[2].cpu().numpy().view(np.uint32)
        dead_blocks = 0
        for qt in range(case.L // 128):
            for kt in range(qt):                                                   # off-diagonal tiles: a key is dead iff it expired before the tile's rows
                if (bmp[0, 0, qt, kt // 32] >> np.uint32(kt % 32)) & np.uint32(1):
                    blk = (e[0, 0, kt * 128:(kt + 1) * 128].reshape(8, 16) <= qt * 128).all(1)
                    dead_blocks += int(blk.sum())
        assert dead_blocks > 0, case.name
        for path in (dma.DMA_FLAG_TILE_PATH, dma.DMA_FLAG_COMPACT_KV):
            outs = []
            for extra in (dma.DMA_FLAG_BLOCK_SKIP, 0):
                p = problem_of(case, flags=path | extra)
                ws = torch.empty(dma.dma_query_workspace(p)[1], dtype=torch.uint8, device=dev)
                outs.append(dma.dma_attn_fwd(p, Q, K, V, *mask, ws=ws))
                assert dma.dma_read_status(ws) == 0
            assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]), (case.name, path)


def test_largest_supported_lengths():
    """The longest sequences the tensor-core kernels take: L = 131072 (1024 key tiles, the forward schedule's capacity; with
    a group of 4 query heads per KV head also the capacity of the backward's step list), forward and backward, tile path and
    token-compacted. Sampled rows and keys against the oracle, dQ on rows where the mask drops keys."""
    case = wl.small(wl.CONFIGS["3"], B=1, Hq=4, Hkv=1, L=131072, w=2048, backward=True, name="max L")
    inp = wl.make_inputs(case)
    ref = Samples(case, inp, nrows=8, nkeys=4)
    got = gpu_run(case, inp, stored=ref.stored, flags=dma.DMA_FLAG_TILE_PATH)
    ref.check(got)
    ref.check(gpu_run(case, inp, stored=ref.stored, flags=dma.DMA_FLAG_COMPACT_KV), "compact ")
    with pytest.raises(dma.DmaError) as e:                        # one tile more is refused, not mis-executed
        too_long = wl.small(case, L=131072 + 128)
        dma.dma_attn_fwd(problem_of(too_long, flags=dma.DMA_FLAG_TILE_PATH), got["O"], got["O"], got["O"], got["bias"], got["expiry"], got["bitmap"])
    assert e.value.status == -4
    with pytest.raises(dma.DmaError) as e:                        # eight heads per KV head at this length: the tile path's step list is too short
        wide = problem_of(wl.small(case, Hq=8), flags=dma.DMA_FLAG_TILE_PATH)
        ws = torch.empty(dma.dma_query_workspace(wide)[2], dtype=torch.uint8, device="cuda:0")
        dma.dma_attn_bwd(wide, got["O"], got["O"], got["O"], got["O"], got["O"], got["lse"], got["bias"], got["expiry"], got["bitmap"], ws=ws)
    assert e.value.status == -4


def test_whole_step_can_be_captured_in_a_cuda_graph():
    """The stream entry points only enqueue work (no allocation, no synchronisation): mask build, forward and backward are
    captured once and replayed; the replay reproduces the eager results."""
    dev = torch.device("cuda:0")
    case = wl.small(C2, B=1, Hq=8, Hkv=2, L=1024, w=256, backward=True, name="graph")
    inp = wl.make_inputs(case)
    eager = gpu_run(case, inp)
    p = problem_of(case)
    Q, K, V, dO = (inp[k].to(dev) for k in ("Q", "K", "V", "dO"))
    W, A = inp["W_delta"].to(dev), inp["A"].to(dev)
    m_ws, f_ws, b_ws = (torch.empty(n, dtype=torch.uint8, device=dev) for n in dma.dma_query_workspace(p))
    bias, expiry, bitmap = (torch.empty_like(eager[k]) for k in ("bias", "expiry", "bitmap"))
    O, lse = torch.empty_like(eager["O"]), torch.empty_like(eager["lse"])
    dQ, dK, dV, dM = (torch.empty_like(eager[k]) for k in ("dQ", "dK", "dV", "dM"))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        dma.dma_mask_build(p, V, W, A, bias, expiry, bitmap, m_ws)
        dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap, O, lse, f_ws)
        dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, b_ws)
    for _ in range(2):
        for t in (bias, expiry, bitmap, O, lse, dQ, dK, dV, dM):
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert dma.dma_read_status(f_ws) == 0 and dma.dma_read_status(b_ws) == 0
        for k, t in (("bias", bias), ("expiry", expiry), ("bitmap", bitmap), ("O", O), ("lse", lse), ("dK", dK), ("dV", dV)):
            assert torch.equal(t, eager[k]), k
        assert_close(dQ, f64(eager["dQ"]), case.dtype, "dQ (replayed)")        # atomics: order-dependent rounding
        assert_close(dM, f64(eager["dM"]), case.dtype, "dM (replayed)")


def test_bounded_wait_reports_timeout_and_context_survives():
    # a wait that nothing satisfies gives up after its limit and leaves a status, instead of hanging the GPU
    dev = torch.device("cuda:0")
    ws = torch.zeros(256, dtype=torch.uint8, device=dev)
    dma.dma_selftest_wait_timeout(ws)
    assert dma.dma_read_status(ws) == -7
    # the context is still usable and a normal call leaves a clean status
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=256, w=64, backward=False, name="after-timeout")
    inp = wl.make_inputs(case)
    got = gpu_run(case, inp, backward=False)
    assert torch.isfinite(got["O"].float()).all()


# ---- token-compacted forward (DMA_FLAG_COMPACT_KV): same results as the oracle, from the gathered key lists ----------

def _compact_run(case, inp):
    dev = torch.device("cuda:0")
    p = problem_of(case)
    pc = problem_of(case, flags=dma.DMA_FLAG_COMPACT_KV)
    Q, K, V = (inp[k].to(dev) for k in ("Q", "K", "V"))
    bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(dev), inp["A"].to(dev))
    ws = torch.empty(dma.dma_query_workspace(pc)[1], dtype=torch.uint8, device=dev)
    O, lse = dma.dma_attn_fwd(pc, Q, K, V, bias, expiry, bitmap, ws=ws)
    torch.cuda.synchronize()
    assert dma.dma_read_status(ws) == 0
    return {"bias": bias, "expiry": expiry, "bitmap": bitmap, "O": O, "lse": lse}


@pytest.mark.parametrize("kw", [
    dict(B=1, Hq=2, Hkv=1, L=384, w=64),            # ragged pair count (3 query tiles), small window
    dict(B=2, Hq=4, Hkv=2, L=1000, w=200),          # ragged tail rows, GQA
    dict(B=1, Hq=2, Hkv=2, L=1536, w=2000),         # w >= L: every causal key is gathered (dense causal attention)
    dict(B=1, Hq=4, Hkv=1, L=2048, w=1),            # w = 1: one key per row
])
def test_compact_forward_small_cases(kw):
    case = wl.small(C2, name="compact-small", backward=False, **kw)
    inp = wl.make_inputs(case)
    got = _compact_run(case, inp)
    dl, e, _ = oracle_mask(case, inp)                     # the oracle's own mask, not the GPU's
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    ref = oracle.forward(inp["Q"].double().numpy(), inp["K"].double().numpy(), inp["V"].double().numpy(),
                         dl.astype(np.float64), expiry=e, scale=case.d ** -0.5)
    assert_close(got["O"], ref[0], case.dtype, "compact O")
    assert_close(got["lse"], ref[1], case.dtype, "compact lse", lse=True)


@pytest.mark.parametrize("key", ["3", "S", "5"])
def test_compact_forward_full_size_sampled(key):
    case = wl.CONFIGS[key]
    inp = wl.make_inputs(case)
    Samples(case, inp, forward_only=True).check(_compact_run(case, inp), "compact ")


def test_compact_flag_is_rejected_where_unsupported():
    dev = torch.device("cuda:0")
    for case in (wl.small(C1, B=1, Hq=2, Hkv=1, L=256, w=64, d=128, name="compact-fp32"),
                 wl.small(C2, B=1, Hq=2, Hkv=1, L=256, w=64, d=64, name="compact-d64-cuda-cores")):
        inp = wl.make_inputs(case)
        flags = dma.DMA_FLAG_COMPACT_KV | (dma.DMA_FLAG_SIMT if case.dtype == "bf16" else 0)
        with pytest.raises(dma.DmaError) as e:
            gpu_run(case, inp, backward=False, flags=flags)
        assert e.value.status == -4


def test_bf16_d64_runs_on_the_tensor_core_kernels():
    """bf16 with 64 channels runs on the d = 64 instantiations of the tensor-core kernels (both paths): results against the
    oracle within the gate, on strided inputs too, nothing written outside the views."""
    dev = torch.device("cuda:0")
    case = wl.small(C2, B=2, Hq=4, Hkv=2, L=700, w=96, d=64, backward=True, name="d64-native")
    inp = wl.make_inputs(case)
    dl, e, _ = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    st = stored_forward(case, ref["O"], ref["lse"])
    for flags in (0, dma.DMA_FLAG_COMPACT_KV):
        compare(case, gpu_run(case, inp, stored=st, flags=flags), ref)
    # strided Q / K / V / O views of wider buffers
    big = {k: torch.randn(case.B, case.L + 9, (case.Hq if k in ("Q", "dO") else case.Hkv) + 1, 64).to(case.torch_dtype).to(dev) for k in ("Q", "K", "V", "dO")}
    view = {k: big[k][:, 3:3 + case.L, 1:] for k in big}
    for k in view:
        view[k].copy_(inp[k].to(dev))
    p = problem_of(case)
    for sdst, t in ((p.q_stride, view["Q"]), (p.k_stride, view["K"]), (p.v_stride, view["V"]), (p.o_stride, view["dO"])):
        sdst[0], sdst[1], sdst[2] = t.stride(0), t.stride(1), t.stride(2)
    bias, expiry, bitmap = dma.dma_mask_build(p, view["V"], inp["W_delta"].to(dev), inp["A"].to(dev))
    Obuf = torch.zeros_like(big["dO"])
    O, lse = dma.dma_attn_fwd(p, view["Q"], view["K"], view["V"], bias, expiry, bitmap, O=Obuf[:, 3:3 + case.L, 1:])
    dQb, dKb, dVb = torch.zeros_like(big["Q"]), torch.zeros_like(big["K"]), torch.zeros_like(big["V"])
    Oin = torch.zeros_like(big["dO"])[:, 3:3 + case.L, 1:]                       # the oracle's stored O in the same strided layout
    Oin.copy_(torch.from_numpy(st["O"]).to(case.torch_dtype).to(dev))
    dQ, dK, dV, dM = dma.dma_attn_bwd(p, view["Q"], view["K"], view["V"], Oin, view["dO"], torch.from_numpy(st["lse"]).to(dev), bias, expiry, bitmap,
                                      dQ=dQb[:, 3:3 + case.L, 1:], dK=dKb[:, 3:3 + case.L, 1:], dV=dVb[:, 3:3 + case.L, 1:])
    torch.cuda.synchronize()
    compare(case, {"O": O, "lse": lse, "dQ": dQ, "dK": dK, "dV": dV, "dM": dM}, ref)
    assert float(Obuf[:, :3].abs().max()) == 0.0 and float(Obuf[:, :, 0].abs().max()) == 0.0
    assert float(dKb[:, :3].abs().max()) == 0.0 and float(dKb[:, :, 0].abs().max()) == 0.0


def test_compact_kernels_on_strided_k_and_v():
    """K and V living inside larger buffers (spare sequence capacity, extra heads between the used ones): the gathers follow
    the descriptor's strides; results equal those on packed copies of the same data."""
    dev = torch.device("cuda:0")
    case = wl.small(C2, B=2, Hq=4, Hkv=2, L=700, w=96, backward=True, name="compact-strided")
    inp = wl.make_inputs(case)
    ref = gpu_run(case, inp, flags=dma.DMA_FLAG_COMPACT_KV)
    B, L, Hkv, d = case.B, case.L, case.Hkv, case.d
    cap, Hbig = L + 52, 2 * Hkv + 1
    bigK = torch.randn(B, cap, Hbig, d).to(case.torch_dtype).to(dev)
    bigV = torch.randn(B, cap, Hbig, d).to(case.torch_dtype).to(dev)
    Kv, Vv = bigK[:, :L, 1:1 + 2 * Hkv:2], bigV[:, :L, 1:1 + 2 * Hkv:2]          # every other head, starting at head 1
    Kv.copy_(inp["K"].to(dev)); Vv.copy_(inp["V"].to(dev))
    p = problem_of(case, flags=dma.DMA_FLAG_COMPACT_KV)
    for sdst, t in ((p.k_stride, Kv), (p.v_stride, Vv)):
        sdst[0], sdst[1], sdst[2] = t.stride(0), t.stride(1), t.stride(2)
    Q, dO = inp["Q"].to(dev), inp["dO"].to(dev)
    O, lse = dma.dma_attn_fwd(p, Q, Kv, Vv, ref["bias"], ref["expiry"], ref["bitmap"])
    dK, dV = torch.zeros_like(bigK), torch.zeros_like(bigV)
    dKv, dVv = dK[:, :L, 1:1 + 2 * Hkv:2], dV[:, :L, 1:1 + 2 * Hkv:2]
    dQ, _, _, dM = dma.dma_attn_bwd(p, Q, Kv, Vv, O, dO, lse, ref["bias"], ref["expiry"], ref["bitmap"], dK=dKv, dV=dVv)
    torch.cuda.synchronize()
    assert torch.equal(O, ref["O"]) and torch.equal(lse, ref["lse"])
    assert_close(dKv, f64(ref["dK"]), case.dtype, "dK (strided)")
    assert_close(dVv, f64(ref["dV"]), case.dtype, "dV (strided)")
    assert_close(dQ, f64(ref["dQ"]), case.dtype, "dQ (strided)")
    assert_close(dM, f64(ref["dM"]), case.dtype, "dM (strided)")
    untouched = torch.ones(Hbig, dtype=torch.bool); untouched[1:1 + 2 * Hkv:2] = False
    assert float(dK[:, :, untouched].abs().max()) == 0.0 and float(dK[:, L:].abs().max()) == 0.0


# ---- token-compacted backward (DMA_FLAG_COMPACT_KV): key tiles follow a lifetime-sorted permutation per query head -----

@pytest.mark.parametrize("case", [c for c in CASES if c.dtype == "bf16" and c.d == 128], ids=lambda c: c.name)
def test_compact_backward_small_cases(case):
    # the same small cases as the tile path (ragged tails and padding entries in the permutation, several query heads
    # adding into one KV head, w = 1 where almost every key is never kept, w >= L where nothing expires, peaked scores)
    inp = wl.make_inputs(case)
    dl, e, _ = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    got = gpu_run(case, inp, stored=stored_forward(case, ref["O"], ref["lse"]), flags=dma.DMA_FLAG_COMPACT_KV)
    assert np.array_equal(got["expiry"].cpu().numpy(), e)
    compare(case, got, ref)


def test_compact_backward_deterministic_option():
    """DMA_FLAG_DETERMINISTIC: the query heads of a group write dK / dV contributions to accumulators of their own, added in
    head order: the same bits from run to run (four heads per KV head here), and the same parity with the oracle."""
    case = wl.small(C2, B=2, Hq=8, Hkv=2, L=1100, w=150, backward=True, name="compact deterministic")
    inp = wl.make_inputs(case)
    dl, e, _ = oracle_mask(case, inp)
    ref = oracle_all(case, inp, dl, e)
    st = stored_forward(case, ref["O"], ref["lse"])
    flags = dma.DMA_FLAG_COMPACT_KV | dma.DMA_FLAG_DETERMINISTIC
    runs = [gpu_run(case, inp, stored=st, flags=flags) for _ in range(3)]
    compare(case, runs[0], ref)
    for r in runs[1:]:
        assert torch.equal(r["dK"], runs[0]["dK"]) and torch.equal(r["dV"], runs[0]["dV"])
    plain = gpu_run(case, inp, stored=st, flags=dma.DMA_FLAG_COMPACT_KV)
    assert_close(plain["dK"], f64(runs[0]["dK"]), case.dtype, "dK (atomic against ordered sums)")
    assert dma.dma_query_workspace(problem_of(case, flags=flags))[2] > dma.dma_query_workspace(problem_of(case, flags=dma.DMA_FLAG_COMPACT_KV))[2]


@pytest.mark.parametrize("key", ["3", "4w256", "4w2048", "S"])
def test_compact_backward_full_size_sampled(key):
    case = wl.CONFIGS[key]
    inp = wl.make_inputs(case)
    ref = Samples(case, inp)
    ref.check(gpu_run(case, inp, stored=ref.stored, flags=dma.DMA_FLAG_COMPACT_KV), "compact ")
