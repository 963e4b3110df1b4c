"""GPU parity of mask generation (Sec. 4.1) against the CPU oracle: delta, expiry and bitmap bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import workloads as wl

from helpers import bits_equal, gpu_mask, oracle_mask

pytestmark = pytest.mark.gpu

C1, C2 = wl.CONFIGS["1"], wl.CONFIGS["2"]
SMALL = [
    C1,
    wl.small(C1, L=1, w=1, name="L1"),
    wl.small(C1, L=77, w=200, name="w>=L ragged"),
    wl.small(C1, L=300, w=1, name="w=1"),
    wl.small(C1, d=128, Hq=4, Hkv=2, L=513, w=100, name="fp32 d128 gqa"),
    wl.small(C2, B=2, Hq=4, Hkv=2, L=1000, w=129, name="bf16 ragged"),
    wl.small(C2, B=1, Hq=8, Hkv=2, L=2048, w=256, d=64, name="bf16 d64"),
    wl.small(C2, B=1, Hq=6, Hkv=1, L=777, w=300, name="bf16 group of 6"),
]


def check_mask(case, inp, tile=(128, 128), **kw):
    p, bias, expiry, bitmap = gpu_mask(case, inp, **kw)
    dl, e, bmp = oracle_mask(case, inp, tile)
    assert bits_equal(bias, dl), "delta bits differ"
    assert np.array_equal(expiry.cpu().numpy(), e), "expiry differs"
    assert np.array_equal(bitmap.cpu().numpy().view(np.uint32), bmp), "bitmap differs"
    return e, bmp


@pytest.mark.parametrize("case", SMALL, ids=lambda c: c.name)
def test_mask_small_cases(case):
    e, _ = check_mask(case, wl.make_inputs(case))
    i = np.arange(case.L)
    kept_per_row = ((e[..., None, :] > i[:, None]) & (i[None, :] <= i[:, None])).sum(-1)
    assert (kept_per_row == np.minimum(case.w, i + 1)).all()          # exactly min(w, visible) keys per row


def test_mask_heavy_ties():
    # duplicated value rows give exactly equal delta: ties must go to the lower index
    case = wl.small(C2, B=1, Hq=4, Hkv=2, L=1500, w=200, name="ties")
    inp = wl.make_inputs(case)
    inp["V"] = inp["V"][:, torch.arange(case.L) % 37]
    check_mask(case, inp)
    inp["V"] = torch.zeros_like(inp["V"])                               # all equal: keys 0..w-1 ("sink")
    e, _ = check_mask(case, inp)
    assert (e[..., :200] == case.L).all() and (e[..., 200:] == np.arange(200, case.L)).all()


@pytest.mark.parametrize("L,w", [(300_001, 5000), (4097, 64), (8192 + 256, 300), (131_072, 131_071)])
def test_mask_long_heads_with_ragged_run_counts(L, w):
    """The selection merges sorted runs level by level; a length that is not a power of two leaves a trailing run without
    a partner on some levels (300 001 keys: 1172 chunks, 19 levels). Every expiry and the bitmap against the oracle."""
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=L, w=w, d=64, name="long")
    g = torch.Generator().manual_seed(L)
    inp = {"V": torch.randn(case.B, case.L, case.Hkv, case.d, generator=g).to(case.torch_dtype),
           "W_delta": torch.randn(case.Hq, case.d, generator=g) / 8.0, "A": torch.rand(case.Hq, generator=g) * 1.5 + 0.5}
    inp["V"][:, L // 3: L // 3 + 700] = inp["V"][:, :1]                 # a run of exactly equal delta across chunk boundaries
    check_mask(case, inp)


def test_mask_other_tile_sizes():
    case = wl.small(C2, B=1, Hq=2, Hkv=1, L=900, w=64, name="tiles")
    inp = wl.make_inputs(case)
    for tm, tn in ((64, 64), (64, 128), (128, 64), (32, 256)):
        check_mask(case, inp, (tm, tn), tile_m=tm, tile_n=tn)


def test_delta_bits_on_a_million_preactivations():
    # V = z * e_0 and W = e_0 make the projection exact (z = fma(z, 1, 0)), so the whole fp32 range of
    # pre-activations can be pushed through softplus/exp and compared bit for bit.
    B, L, H, d = 16, 65536, 1, 64
    g = torch.Generator().manual_seed(5)
    z = torch.randn(B, L, generator=g) * 3
    edge = torch.tensor([0.0, -0.0, 1e-30, -1e-30, 20.0, -20.0, 86.9, -86.9, 0.34657359, -0.34657359, 1e-7, 40.0, -40.0])
    z[0, : len(edge)] = edge
    z[1] = torch.linspace(-25, 25, L)
    z[2] = (torch.arange(L) - L // 2).float() * 0.34657359 * 2 / 64       # straddles the n-rounding boundaries of exp
    V = torch.zeros(B, L, H, d)
    V[..., 0] = z[:, :, None]
    W = torch.zeros(H, d)
    W[:, 0] = 1.0
    case = wl.Case("zsweep", B, H, H, L, d, L, "fp32")
    for a in (0.5, 1.37, 2.0):
        inp = {"V": V, "W_delta": W, "A": torch.full((H,), a)}
        p, bias, expiry, bitmap = gpu_mask(case, inp)
        zz, dl = oracle.delta(V.numpy(), W.numpy(), inp["A"].numpy(), H)
        assert np.array_equal(zz[:, 0], z.numpy())
        assert bits_equal(bias, dl)


@pytest.mark.parametrize("key", ["2", "3", "4w256", "4w8192", "5", "S"])
def test_mask_full_size_configs(key):
    case = wl.CONFIGS[key]
    e, bmp = check_mask(case, wl.make_inputs(case))
    assert (e >= np.arange(case.L)).all()
