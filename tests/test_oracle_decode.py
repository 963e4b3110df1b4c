"""Pins for the oracle's decoding step: it must equal the last row of the (separately pinned) full-sequence forward,
dense softmax attention when w >= N, and a single key when w = 1."""
import numpy as np

import oracle


def _case(seed, B=2, N=37, Hq=4, Hkv=2, d=8):
    r = np.random.default_rng(seed)
    return (r.standard_normal((B, Hq, d)), r.standard_normal((B, N, Hkv, d)), r.standard_normal((B, N, Hkv, d)),
            np.exp(r.standard_normal((B, Hq, N))).astype(np.float32))


def test_equals_last_row_of_the_training_forward():
    # the last query row of a causal sequence sees every key; its top-w set is the decode step's selection
    q, K, V, delta = _case(1)
    B, N, Hq, w = q.shape[0], K.shape[1], q.shape[1], 9
    Q = np.zeros((B, N, Hq, q.shape[2])); Q[:, -1] = q
    e = oracle.select_expiry(delta, w)
    O, lse = oracle.forward(Q, K, V, delta.astype(np.float64), expiry=e, rows=np.array([N - 1], np.int32))
    o, l, idx = oracle.decode(q, K, V, delta, w)
    assert np.allclose(o, O[:, 0]) and np.allclose(l, lse[:, :, 0])
    kept = oracle.keep_from_expiry(e)[:, :, N - 1, :]                      # [B, Hq, N] keys kept by the last row
    for b in range(B):
        for h in range(Hq):
            assert np.array_equal(np.flatnonzero(kept[b, h]), idx[b, h])


def test_window_covering_everything_is_dense_attention():
    q, K, V, delta = _case(2)
    o, l, idx = oracle.decode(q, K, V, delta, 1000)
    B, Hq, d = q.shape
    for b in range(B):
        for h in range(Hq):
            s = K[b, :, h // 2, :] @ q[b, h] / np.sqrt(d) + delta[b, h]
            p = np.exp(s - s.max()); p /= p.sum()
            assert np.allclose(o[b, h], p @ V[b, :, h // 2, :])
            assert np.isclose(l[b, h], np.log(np.exp(s - s.max()).sum()) + s.max())
            assert np.array_equal(idx[b, h], np.arange(K.shape[1]))


def test_window_of_one_returns_the_argmax_key_and_ties_go_to_the_lower_index():
    q, K, V, delta = _case(3)
    delta[:, :, :] = 1.0                       # all tied: index 0 wins
    delta[0, 1, 20] = 5.0; delta[0, 1, 30] = 5.0          # tie at the top: 20 wins
    o, l, idx = oracle.decode(q, K, V, delta, 1)
    assert idx[0, 1, 0] == 20 and (np.delete(idx[:, :, 0].ravel(), 1) == 0).all()
    assert np.allclose(o[0, 1], V[0, 20, 0]) and np.allclose(o[1, 3], V[1, 0, 1])
    o3, _, idx3 = oracle.decode(q, K, V, delta, 3)
    assert list(idx3[0, 1]) == [0, 20, 30] and list(idx3[1, 0]) == [0, 1, 2]
