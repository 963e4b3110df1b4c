"""Pins for the oracle's non-causal mode (the App. A listing with an all-zero causal mask: every row of a head keeps
the same top-w keys): brute force from the definition, dense softmax attention for w >= L, the last causal row, the
separately pinned decoding step, and finite differences of an independently written forward."""
import numpy as np

import oracle


def _case(seed, B=1, L=13, Hq=2, Hkv=1, d=8):
    r = np.random.default_rng(seed)
    return (r.standard_normal((B, L, Hq, d)), r.standard_normal((B, L, Hkv, d)), r.standard_normal((B, L, Hkv, d)),
            np.exp(r.standard_normal((B, Hq, L))).astype(np.float32), r.standard_normal((B, L, Hq, d)))


def _dense_forward(Q, K, V, bias, keepcols, scale):
    """softmax(Q K^T scale + bias) V over the listed key columns (per batch and head), straight numpy."""
    B, L, Hq, d = Q.shape
    G = Hq // K.shape[2]
    O = np.zeros_like(Q); lse = np.zeros((B, Hq, L))
    for b in range(B):
        for h in range(Hq):
            cols = keepcols[b][h]
            s = Q[b, :, h] @ K[b, cols, h // G].T * scale + bias[b, h, cols][None, :]
            m = s.max(-1, keepdims=True)
            p = np.exp(s - m)
            lse[b, h] = (m + np.log(p.sum(-1, keepdims=True)))[:, 0]
            O[b, :, h] = (p / p.sum(-1, keepdims=True)) @ V[b, cols, h // G]
    return O, lse


def test_selection_is_the_top_w_of_the_whole_head():
    r = np.random.default_rng(1)
    dl = np.exp(r.standard_normal((2, 3, 40))).astype(np.float32)
    dl[0, 0, [3, 17, 30]] = dl[0, 0].max()                       # ties at the top: lower index first
    dl[1, 2, :] = 1.0                                             # all tied
    for w in (1, 2, 7, 40, 99):
        e = oracle.select_noncausal(dl, w)
        for b in range(2):
            for h in range(3):
                want = sorted(range(40), key=lambda j: (-float(dl[b, h, j]), j))[:w]
                assert sorted(np.nonzero(e[b, h])[0].tolist()) == sorted(want)
                assert set(e[b, h].tolist()) <= {0, 40}
        keep = oracle.keep_from_expiry_noncausal(e)
        assert (keep == (e[..., None, :] > 0)).all()              # the same set for every row


def test_forward_is_dense_attention_over_the_kept_columns():
    Q, K, V, dl, _ = _case(2)
    L, d = Q.shape[1], Q.shape[3]
    for w in (4, L, 50):
        e = oracle.select_noncausal(dl, w)
        O, lse = oracle.forward(Q, K, V, dl, expiry=e, causal=False)
        cols = [[np.nonzero(e[b, h])[0] for h in range(Q.shape[2])] for b in range(Q.shape[0])]
        Od, lsed = _dense_forward(Q, K, V, dl.astype(np.float64), cols, d ** -0.5)
        assert np.allclose(O, Od) and np.allclose(lse, lsed)
    # the keep-matrix form agrees with the interval form
    e = oracle.select_noncausal(dl, 4)
    O1, l1 = oracle.forward(Q, K, V, dl, expiry=e, causal=False)
    O2, l2 = oracle.forward(Q, K, V, dl, keep=oracle.keep_from_expiry_noncausal(e), causal=False)
    assert np.array_equal(O1, O2) and np.array_equal(l1, l2)


def test_last_row_equals_the_causal_last_row_and_the_decoding_step():
    Q, K, V, dl, _ = _case(3, L=21, Hq=4, Hkv=2)
    w = 6
    On, ln = oracle.forward(Q, K, V, dl, expiry=oracle.select_noncausal(dl, w), causal=False)
    Oc, lc = oracle.forward(Q, K, V, dl, expiry=oracle.select_expiry(dl, w))
    assert np.allclose(On[:, -1], Oc[:, -1]) and np.allclose(ln[..., -1], lc[..., -1])
    o, lse, _ = oracle.decode(Q[:, -1], K, V, dl, w)
    assert np.allclose(On[:, -1], o) and np.allclose(ln[..., -1], lse)


def test_backward_matches_central_differences():
    Q, K, V, dl, dO = _case(4, L=9, Hq=2, Hkv=1, d=4)
    bias = dl.astype(np.float64)
    e = oracle.select_noncausal(dl, 4)
    cols = [[np.nonzero(e[b, h])[0] for h in range(2)] for b in range(1)]
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias, expiry=e, causal=False)
    loss = lambda Q_, K_, V_, b_: float((dO * _dense_forward(Q_, K_, V_, b_, cols, 4 ** -0.5)[0]).sum())
    eps = 1e-6
    r = np.random.default_rng(5)
    for X, g, slot in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2), (bias, dM, 3)):
        for _ in range(10):
            idx = tuple(r.integers(0, n) for n in X.shape)
            args = [Q, K, V, bias]
            Xp, Xm = X.copy(), X.copy(); Xp[idx] += eps; Xm[idx] -= eps
            args[slot] = Xp; fp = loss(*args)
            args[slot] = Xm; fm = loss(*args)
            assert abs((fp - fm) / (2 * eps) - g[idx]) < 1e-5 * max(1.0, abs(g[idx])), (slot, idx)
    # a key that is not selected gets no gradient at all
    dead = np.nonzero(e[0, 0] == 0)[0]
    assert np.all(dM[0, 0, dead] == 0)


def test_keys_subset_and_rows_subset_agree_with_the_full_result():
    Q, K, V, dl, dO = _case(6, L=17, Hq=2, Hkv=2)
    e = oracle.select_noncausal(dl, 5)
    O, lse = oracle.forward(Q, K, V, dl, expiry=e, causal=False)
    rows = np.array([0, 3, 16], np.int32)
    Or, lr = oracle.forward(Q, K, V, dl, expiry=e, rows=rows, causal=False)
    assert np.allclose(O[:, rows], Or) and np.allclose(lse[..., rows], lr)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, dl, expiry=e, causal=False)
    keys = np.array([1, 9, 16], np.int32)
    _, dKk, dVk, dMk = oracle.backward(Q, K, V, dO, dl, expiry=e, keys=keys, want_dq=False, causal=False)
    assert np.allclose(dK[:, keys], dKk) and np.allclose(dV[:, keys], dVk) and np.allclose(dM[..., keys], dMk)
