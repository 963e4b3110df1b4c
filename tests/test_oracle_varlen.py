"""Pins for the oracle's packed-sequence (variable-length) selection: brute force from the definition on small
inputs, and the packed attention equal to the attention of every sequence on its own."""
import numpy as np

import oracle


def _brute_keep(dl, w, cu):
    """keep[i, j] straight from the definition: row i sees the keys of its own sequence up to itself, orders them by
    (delta descending, index ascending) and keeps the first w."""
    L = dl.shape[-1]
    keep = np.zeros((L, L), np.uint8)
    for s0, s1 in zip(cu, cu[1:]):
        for i in range(s0, s1):
            vis = sorted(range(s0, i + 1), key=lambda j: (-float(dl[j]), j))
            for j in vis[:w]:
                keep[i, j] = 1
    return keep


def test_matches_brute_force_definition():
    r = np.random.default_rng(1)
    for cu, w in (([0, 5, 6, 20, 37], 4), ([0, 1, 2, 3], 2), ([0, 33], 7), ([0, 9, 40], 1), ([0, 16, 32], 64)):
        dl = np.exp(r.standard_normal(cu[-1])).astype(np.float32)
        dl[r.integers(0, cu[-1], 6)] = dl[0]                      # ties: the lower index wins
        e = oracle.select_expiry_varlen(dl[None], w, cu)[0]
        assert np.array_equal(oracle.keep_from_expiry(e[None])[0], _brute_keep(dl, w, cu))
        for s0, s1 in zip(cu, cu[1:]):
            assert e[s0:s1].max() <= s1 and e[s0:s1].min() >= s0


def test_single_sequence_is_the_plain_selection():
    r = np.random.default_rng(2)
    dl = np.exp(r.standard_normal((2, 3, 50))).astype(np.float32)
    assert np.array_equal(oracle.select_expiry_varlen(dl, 8, [0, 50]), oracle.select_expiry(dl, 8))


def test_packed_attention_equals_each_sequence_alone():
    r = np.random.default_rng(3)
    cu, w, B, Hq, Hkv, d = [0, 7, 19, 40], 5, 1, 2, 1, 8
    L = cu[-1]
    Q = r.standard_normal((B, L, Hq, d)); K = r.standard_normal((B, L, Hkv, d)); V = r.standard_normal((B, L, Hkv, d))
    dO = r.standard_normal((B, L, Hq, d))
    dl = np.exp(r.standard_normal((B, Hq, L))).astype(np.float32)
    e = oracle.select_expiry_varlen(dl, w, cu)
    O, lse = oracle.forward(Q, K, V, dl, expiry=e)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, dl, expiry=e)
    for s0, s1 in zip(cu, cu[1:]):
        sl = slice(s0, s1)
        es = oracle.select_expiry(dl[..., sl], w)
        Os, lses = oracle.forward(Q[:, sl], K[:, sl], V[:, sl], dl[..., sl], expiry=es)
        assert np.allclose(O[:, sl], Os) and np.allclose(lse[..., sl], lses)
        g = oracle.backward(Q[:, sl], K[:, sl], V[:, sl], dO[:, sl], dl[..., sl], expiry=es)
        for packed, alone in zip((dQ[:, sl], dK[:, sl], dV[:, sl], dM[..., sl]), g):
            assert np.allclose(packed, alone)
