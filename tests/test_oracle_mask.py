"""Pins for the oracle's mask construction (Sec. 4.1): delta, per-row top-w selection, block bitmap.

None of these compares the oracle with itself only: each checks a closed form, an invariant the method
fixes, a library routine on a special case, or the definition evaluated by other means.
"""
import math

import numpy as np
import pytest
import torch

import oracle


def ulp_diff(a, b):
    """Distance in units of the fp32 last place between fp32 array a and fp64 array b."""
    a = np.asarray(a, np.float32)
    b = np.asarray(b, np.float64)
    spacing = np.spacing(np.abs(b).astype(np.float32)).astype(np.float64)
    return np.abs(a.astype(np.float64) - b) / spacing


# ------------------------------------------------------------------------------------------- delta

def test_exp_spec_close_to_libm_over_range():
    xs = np.concatenate([np.linspace(-87, 88, 20001), np.linspace(-1, 1, 2001), [0.0, 1e-8, -1e-8]]).astype(np.float32)
    got = np.array([oracle.exp_spec(x) for x in xs], np.float32)
    assert ulp_diff(got, np.exp(xs.astype(np.float64))).max() <= 2.0
    assert oracle.exp_spec(0.0) == 1.0
    # clamp: arguments beyond the documented range saturate, never overflow or reach zero
    assert oracle.exp_spec(1000.0) == oracle.exp_spec(88.0) and math.isfinite(oracle.exp_spec(88.0))
    assert oracle.exp_spec(-1000.0) == oracle.exp_spec(-87.0) > 0.0


def test_log1p_and_softplus_close_to_libm():
    ts = np.concatenate([np.linspace(1e-6, 1, 5001), np.float32(2.0) ** -np.arange(1, 120)]).astype(np.float32)
    got = np.array([oracle.log1p_spec(t) for t in ts], np.float32)
    assert ulp_diff(got, np.log1p(ts.astype(np.float64))).max() <= 4.0   # the spec asks for "a few ulp", not correct rounding
    zs = np.linspace(-30, 30, 6001).astype(np.float32)
    got = np.array([oracle.softplus_spec(z) for z in zs], np.float32)
    assert ulp_diff(got, np.logaddexp(0.0, zs.astype(np.float64))).max() <= 4.0
    assert oracle.softplus_spec(100.0) == 100.0            # softplus(z) -> z for large z


def test_delta_closed_forms():
    rng = np.random.default_rng(0)
    B, L, Hq, Hkv, d = 2, 16, 4, 2, 64
    W = rng.standard_normal((Hq, d)).astype(np.float32) / 8
    A = rng.uniform(0.5, 2, Hq).astype(np.float32)
    # V = 0  ->  z = 0, softplus = ln 2, delta = exp(A ln 2) = 2^A
    z, dl = oracle.delta(np.zeros((B, L, Hkv, d), np.float32), W, A, Hq)
    assert (z == 0).all()
    assert ulp_diff(dl, np.broadcast_to((2.0 ** A.astype(np.float64))[None, :, None], dl.shape)).max() <= 4
    # A = 0  ->  delta = 1 exactly
    V = rng.standard_normal((B, L, Hkv, d)).astype(np.float32)
    _, dl = oracle.delta(V, W, np.zeros(Hq, np.float32), Hq)
    assert (dl == 1.0).all()
    # V = unit vector e_c in every row  ->  z = W[h, c] exactly
    for c in (0, 7, 8, 37, d - 1):
        V = np.zeros((B, L, Hkv, d), np.float32)
        V[..., c] = 1.0
        z, _ = oracle.delta(V, W, A, Hq)
        assert (z == W[:, c][None, :, None]).all()


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 8, 2), (128, 4, 4)])
def test_delta_matches_fp64_formula_and_gqa_mapping(d, Hq, Hkv):
    rng = np.random.default_rng(d + Hq)
    B, L = 2, 300
    V = rng.standard_normal((B, L, Hkv, d)).astype(np.float32)
    W = (rng.standard_normal((Hq, d)) / math.sqrt(d)).astype(np.float32)
    A = rng.uniform(0.5, 2, Hq).astype(np.float32)
    z, dl = oracle.delta(V, W, A, Hq)
    G = Hq // Hkv
    Vq = np.repeat(V.astype(np.float64), G, axis=2)                 # query head h reads KV head h // G
    z64 = np.einsum("blhc,hc->bhl", Vq, W.astype(np.float64))
    assert np.abs(z - z64).max() < 2e-6 * math.sqrt(d)
    # given the oracle's own (rounded) z, the rest of the chain is within a few ulp of fp64
    ref = np.exp(A.astype(np.float64)[None, :, None] * np.logaddexp(0.0, z.astype(np.float64)))
    assert ulp_diff(dl, ref).max() <= 16      # the fp32 product A*softplus is rounded once before exp: |x|<=12 -> <=~8 ulp
    assert (dl >= 1.0).all()                  # A > 0, softplus > 0


def test_delta_monotone_in_z():
    # rows are multiples of one direction, so z is an increasing function of the multiplier
    d, L = 64, 2001
    W = np.full((1, d), 0.125, np.float32)
    t = np.linspace(-6, 6, L).astype(np.float32)
    V = (t[:, None] * np.ones(d, np.float32))[None, :, None, :]
    for a in (0.5, 1.0, 2.0):
        z, dl = oracle.delta(V, W, np.array([a], np.float32), 1)
        assert (np.diff(z[0, 0]) >= 0).all() and (np.diff(dl[0, 0]) >= 0).all()
        assert dl[0, 0, -1] > dl[0, 0, 0]


def test_delta_golden_bits():
    """Regression guard on delta-v1's bit patterns (file written by tests/golden/make_delta_golden.py,
    which calls only the oracle). The paper prints no worked example; this guards the spec, not the paper."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "delta_v1_bits.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    for z_hex, a_hex, sp_hex, dl_hex in rows:
        z = np.array([int(z_hex, 16)], np.uint32).view(np.float32)[0]
        a = np.array([int(a_hex, 16)], np.uint32).view(np.float32)[0]
        sp = np.float32(oracle.softplus_spec(z))
        dl = np.float32(oracle.exp_spec(np.float32(a) * sp))
        assert int(sp.view(np.uint32)) == int(sp_hex, 16)
        assert int(dl.view(np.uint32)) == int(dl_hex, 16)


# --------------------------------------------------------------------------------------- selection

def brute_keep(dl, w):
    """The definition with no sort: key j is kept by row i iff fewer than w visible keys beat it."""
    L = len(dl)
    keep = np.zeros((L, L), np.uint8)
    for i in range(L):
        for j in range(i + 1):
            n = sum(1 for k in range(i + 1) if dl[k] > dl[j] or (dl[k] == dl[j] and k < j))
            keep[i, j] = n < w
    return keep


@pytest.mark.parametrize("L,w,levels", [(40, 7, 0), (64, 16, 3), (33, 1, 2), (50, 50, 0), (50, 80, 4), (48, 5, 1)])
def test_selection_definition_vs_brute_force(L, w, levels):
    rng = np.random.default_rng(L * 100 + w)
    dl = rng.uniform(1, 5, L).astype(np.float32)
    if levels:                                   # heavy ties: only `levels` distinct values
        dl = rng.integers(1, levels + 1, L).astype(np.float32)
    keep = oracle.select_definition(dl, w)
    assert (keep == brute_keep(dl, w)).all()
    e = oracle.select_expiry(dl, w)
    assert (oracle.keep_from_expiry(e) == keep).all()


def test_selection_matches_topk_without_ties():
    # the App. A listing: causal fill with -inf, then topk per row (distinct values -> unique answer)
    g = torch.Generator().manual_seed(3)
    L, w = 96, 20
    dl = torch.rand(3, L, generator=g).add(1.0)
    m = dl[:, None, :].expand(-1, L, -1).clone()
    causal = torch.ones(L, L).triu(1).bool()
    m.masked_fill_(causal, -float("inf"))
    idx = torch.topk(m, w, dim=-1).indices
    active = torch.zeros(3, L, L).scatter(-1, idx, 1.0)
    active.masked_fill_(causal, 0.0)             # topk picks -inf entries when fewer than w are visible
    keep = oracle.select_definition(dl.numpy(), w)
    assert (keep == active.numpy().astype(np.uint8)).all()


@pytest.mark.parametrize("L,w", [(257, 31), (300, 64), (128, 200), (500, 1)])
def test_selection_invariants_and_interval_form(L, w):
    rng = np.random.default_rng(L + w)
    dl = np.stack([rng.uniform(1, 9, L), rng.integers(1, 4, L), np.round(rng.uniform(1, 3, L), 1)]).astype(np.float32)
    keep = oracle.select_definition(dl, w)
    e = oracle.select_expiry(dl, w)
    assert (oracle.keep_from_expiry(e) == keep).all()
    i = np.arange(L)
    assert (keep.sum(-1) == np.minimum(w, i + 1)[None]).all()          # exactly min(w, visible) keys per row
    assert (np.triu(keep, 1) == 0).all()                               # causal
    nxt, cur = keep[:, 1:, :].astype(int), keep[:, :-1, :].astype(int)
    newcomer = np.zeros_like(nxt)
    newcomer[:, np.arange(L - 1), np.arange(1, L)] = 1
    assert ((nxt - cur - newcomer) <= 0).all()                         # I_{i+1} is inside I_i + {i+1}
    assert (e >= i[None]).all() and (e <= L).all()


def test_selection_special_cases():
    L, w = 200, 17
    i = np.arange(L)
    tri = (i[None, :] <= i[:, None])
    # constant delta: every tie goes to the lower index -> keys 0..w-1
    keep = oracle.select_definition(np.ones(L, np.float32), w)
    assert (keep == (tri & (i[None, :] < w))).all()
    # strictly increasing delta: the w most recent keys (sliding window)
    keep = oracle.select_definition(np.linspace(1, 2, L).astype(np.float32), w)
    assert (keep == (tri & (i[None, :] > i[:, None] - w))).all()
    # strictly decreasing delta: the first w keys
    keep = oracle.select_definition(np.linspace(2, 1, L).astype(np.float32), w)
    assert (keep == (tri & (i[None, :] < w))).all()
    # w >= L: everything visible is kept; expiry = L everywhere
    rnd = np.random.default_rng(1).uniform(1, 2, L).astype(np.float32)
    for ww in (L, L + 5):
        assert (oracle.select_definition(rnd, ww) == tri).all()
        assert (oracle.select_expiry(rnd, ww) == L).all()
    # w = 1: the running first arg-max
    keep = oracle.select_definition(rnd, 1)
    run = np.array([np.argmax(rnd[: t + 1]) for t in range(L)])
    assert (keep.argmax(-1) == run).all() and (keep.sum(-1) == 1).all()


def test_expiry_large_against_running_threshold():
    """At a size where the per-row sort is too slow, the interval form is checked against an independent
    statement: row i keeps key j iff (delta_j, -j) is at least the w-th best of the prefix, found with
    numpy's partition on exact integer keys."""
    rng = np.random.default_rng(7)
    L, w = 3000, 211
    dl = np.round(rng.uniform(1, 30, L), 2).astype(np.float32)        # many ties
    e = oracle.select_expiry(dl, w)
    key = (dl.view(np.uint32).astype(np.int64) << 32) | (0xFFFFFFFF - np.arange(L, dtype=np.int64))
    for i in list(range(0, L, 97)) + [L - 1]:
        pref = key[: i + 1]
        thr = np.partition(pref, len(pref) - w)[len(pref) - w] if i + 1 > w else pref.min()
        assert ((e[: i + 1] > i) == (pref >= thr)).all()


# ------------------------------------------------------------------------------------------ bitmap

def test_bitmap_definition_vs_numpy_and_expiry_form():
    rng = np.random.default_rng(11)
    for L, w, bm, bn in [(300, 40, 64, 64), (256, 64, 128, 128), (200, 9, 32, 64), (130, 130, 128, 128)]:
        dl = np.round(rng.uniform(1, 3, (2, L)), 1).astype(np.float32)
        keep = oracle.select_definition(dl, w)
        e = oracle.select_expiry(dl, w)
        got = oracle.bitmap_definition(keep, bm, bn)
        Tr, Tc = -(-L // bm), -(-L // bn)
        pad = np.zeros((2, Tr * bm, Tc * bn), np.uint8)
        pad[:, :L, :L] = keep
        act = pad.reshape(2, Tr, bm, Tc, bn).any(axis=(2, 4))
        bits = (got[..., np.arange(Tc) // 32] >> (np.arange(Tc) % 32)) & 1
        assert (bits.astype(bool) == act).all()
        assert (oracle.bitmap_from_expiry(e, bm, bn) == got).all()


def test_bitmap_closed_forms():
    L, bm = 1024, 128
    T = L // bm
    t = np.arange(T)
    def unpack(b):
        return ((b[..., t // 32] >> (t % 32)) & 1).astype(bool)
    # w >= L: every causal tile is active, nothing above the diagonal
    e = oracle.select_expiry(np.random.default_rng(0).uniform(1, 2, L).astype(np.float32), L)
    assert (unpack(oracle.bitmap_from_expiry(e, bm, bm)) == (t[None, :] <= t[:, None])).all()
    # increasing delta, w = 128: a band (diagonal tile and the one before it; 129..255 back never reached)
    e = oracle.select_expiry(np.linspace(1, 2, L).astype(np.float32), 128)
    band = (t[None, :] <= t[:, None]) & (t[None, :] >= t[:, None] - 1)
    assert (unpack(oracle.bitmap_from_expiry(e, bm, bm)) == band).all()
    # decreasing delta, w = 128: only the first key tile is ever active
    e = oracle.select_expiry(np.linspace(2, 1, L).astype(np.float32), 128)
    assert (unpack(oracle.bitmap_from_expiry(e, bm, bm)) == (t[None, :] == 0) & (t[:, None] >= 0)).all()
