"""Randomised cross-check of the tensor-core kernels (tile path and token-compacted) against the CUDA-core kernels on the
same masks: random document boundaries, window sizes, head groupings and memory placements. The masks come from the GPU
mask build (checked bit for bit against the oracle elsewhere); what is compared here is kernel against kernel, so that
timing- or placement-dependent defects show up that a single fixed case would miss."""
import numpy as np
import pytest
import torch

from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def one_case(seed):
    r = np.random.default_rng(seed)
    Hkv = int(r.choice([1, 2, 4]))
    G = int(r.choice([1, 2, 4]))
    big = seed >= 16                                               # longer walks: many stage reuses, more documents
    L = int(r.choice([2048, 3000, 4096]) if big else r.choice([384, 512, 640, 900, 1280, 1536]))
    w = int(r.choice([1, 16, 64, 200, 700]))
    d = int(r.choice([64, 128]))
    nseq = int(r.integers(4, 14) if big else r.integers(1, 6))
    cuts = sorted(set(int(c) for c in r.integers(1, L, nseq - 1))) if nseq > 1 else []
    cu = [0] + cuts + [L]
    case = wl.small(wl.CONFIGS["2"], B=int(r.choice([1, 2])), Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, backward=True,
                    seed=1000 + seed, name=f"stress-{seed}")
    return case, cu, int(r.integers(0, 64)) * 0x2468


@pytest.mark.parametrize("seed", range(24))
def test_tensor_core_kernels_equal_the_cuda_core_kernels(seed):
    case, cu, off = one_case(seed)
    inp = wl.make_inputs(case)
    B, L, Hq, Hkv, d = case.B, case.L, case.Hq, case.Hkv, case.d
    nq, nk = B * L * Hq * d, B * L * Hkv * d
    big = torch.empty(2 * nq + 2 * nk + off + 64, dtype=torch.bfloat16, device=DEV)
    o = off
    views = {}
    for k, n, H in (("Q", nq, Hq), ("K", nk, Hkv), ("V", nk, Hkv), ("dO", nq, Hq)):
        views[k] = big[o:o + n].view(B, L, H, d)
        views[k].copy_(inp[k])
        o += n
    Q, K, V, dO = (views[k] for k in ("Q", "K", "V", "dO"))
    W, A = inp["W_delta"].to(DEV), inp["A"].to(DEV)
    cu_t = torch.tensor(cu, dtype=torch.int32, device=DEV)
    mk = lambda flags: dma.problem(B, Hq, Hkv, L, d, case.w, flags=flags)
    p0 = mk(0)
    bias, expiry, bitmap = dma.dma_mask_build_varlen(p0, V, W, A, cu_t)
    ref = None
    for flags in (dma.DMA_FLAG_SIMT, dma.DMA_FLAG_TILE_PATH, dma.DMA_FLAG_COMPACT_KV, 0):
        p = mk(flags)
        O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, bias, expiry, bitmap)
        torch.cuda.synchronize()
        out = {"O": O, "lse": lse, "dQ": dQ, "dK": dK, "dV": dV, "dM": dM}
        assert all(bool(torch.isfinite(t.float()).all()) for t in out.values()), (seed, flags)
        if ref is None:
            ref = out
            continue
        for k, t in out.items():
            a, b = t.float(), ref[k].float()
            scale = max(1.0, float(b.abs().max()))
            tol = (1e-3 if k == "lse" else 4e-2) * scale
            assert float((a - b).abs().max()) <= tol, (seed, flags, k, float((a - b).abs().max()), scale, cu, case)


@pytest.mark.parametrize("seed", range(8))
def test_arbitrary_interval_masks(seed):
    """Any self-consistent (bias, expiry, bitmap) triple is accepted: lifetimes drawn at random (one row, tens of rows,
    hundreds, the whole rest of the sequence) instead of a top-w selection, the bitmap from the oracle's interval rule.
    Every key is kept at least by its own row, so no row is empty."""
    import oracle
    r = np.random.default_rng(100 + seed)
    Hkv, G = int(r.choice([1, 2])), int(r.choice([1, 2, 4]))
    L = int(r.choice([256, 640, 1100]))
    case = wl.small(wl.CONFIGS["2"], B=1, Hq=Hkv * G, Hkv=Hkv, L=L, w=L, d=128, backward=True, seed=2000 + seed, name=f"interval-{seed}")
    inp = wl.make_inputs(case)
    Hq = case.Hq
    kind = r.integers(0, 10, (1, Hq, L))
    life = np.where(kind < 3, 1, np.where(kind < 6, r.integers(1, 64, (1, Hq, L)), np.where(kind < 9, r.integers(64, L + 1, (1, Hq, L)), L)))
    if seed % 2:
        life[:, :, 128:256] = 1                                   # a whole key tile that only its own rows keep
    e = np.minimum(np.arange(L)[None, None, :] + life, L).astype(np.int32)
    bias = r.uniform(0.5, 6.0, (1, Hq, L)).astype(np.float32)
    bitmap = oracle.bitmap_from_expiry(e)
    Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
    bias_t, e_t, bmp_t = torch.from_numpy(bias).to(DEV), torch.from_numpy(e).to(DEV), torch.from_numpy(bitmap.view(np.int32)).to(DEV)
    ref = None
    for flags in (dma.DMA_FLAG_SIMT, dma.DMA_FLAG_TILE_PATH, dma.DMA_FLAG_COMPACT_KV, 0):
        p = dma.problem(1, Hq, Hkv, L, 128, L, flags=flags)
        O, lse = dma.dma_attn_fwd(p, Q, K, V, bias_t, e_t, bmp_t)
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, bias_t, e_t, bmp_t)
        torch.cuda.synchronize()
        out = {"O": O, "lse": lse, "dQ": dQ, "dK": dK, "dV": dV, "dM": dM}
        assert all(bool(torch.isfinite(t.float()).all()) for t in out.values()), (seed, flags)
        if ref is None:
            ref = out
            continue
        for k, t in out.items():
            a, b = t.float(), ref[k].float()
            scale = max(1.0, float(b.abs().max()))
            assert float((a - b).abs().max()) <= (1e-3 if k == "lse" else 4e-2) * scale, (seed, flags, k, float((a - b).abs().max()), scale)


def test_two_host_threads_on_two_streams():
    """The library keeps no state between calls (workspaces are the caller's): two host threads, each on its own stream with
    its own problem and workspaces, get the results of a serial run (O, lse, dK, dV bit for bit; dQ, dM within tolerance)."""
    import threading
    cases = [wl.small(wl.CONFIGS["2"], B=1, Hq=4, Hkv=2, L=1536, w=200, backward=True, seed=71, name="thread-a"),
             wl.small(wl.CONFIGS["2"], B=2, Hq=2, Hkv=1, L=900, w=64, d=64, backward=True, seed=72, name="thread-b")]

    def step(case, inp, flags):
        p = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, flags=flags)
        mask = dma.dma_mask_build(p, inp["V"], inp["W_delta"], inp["A"])
        O, lse = dma.dma_attn_fwd(p, inp["Q"], inp["K"], inp["V"], *mask)
        g = dma.dma_attn_bwd(p, inp["Q"], inp["K"], inp["V"], O, inp["dO"], lse, *mask)
        return dict(zip(("O", "lse", "dQ", "dK", "dV", "dM"), (O, lse) + tuple(g)))

    inps = [{k: v.to(DEV) for k, v in wl.make_inputs(c).items() if isinstance(v, torch.Tensor)} for c in cases]
    serial = [[step(c, i, f) for f in (0, dma.DMA_FLAG_COMPACT_KV)] for c, i in zip(cases, inps)]
    torch.cuda.synchronize()
    errors = []

    def worker(idx):
        try:
            with torch.cuda.stream(torch.cuda.Stream()):
                for rep in range(12):
                    for f, ref in zip((0, dma.DMA_FLAG_COMPACT_KV), serial[idx]):
                        out = step(cases[idx], inps[idx], f)
                        torch.cuda.current_stream().synchronize()
                        for k in ("O", "lse", "dK", "dV"):
                            if not torch.equal(out[k], ref[k]):
                                errors.append((idx, rep, f, k))
                        for k in ("dQ", "dM"):
                            a, b = out[k].float(), ref[k].float()
                            if float((a - b).abs().max()) > 2e-2 * max(1.0, float(b.abs().max())):
                                errors.append((idx, rep, f, k))
        except Exception as ex:                                   # surfaced in the main thread below
            errors.append((idx, repr(ex)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[:5]
