"""Pins for the oracle's full sampling-weight projection (Eq. delta_calc with W mapping all heads' value channels to
one score per head, as the App. A listing's linear layer does) and for its gradient."""
import numpy as np

import oracle


def _case(seed, B=2, L=11, Hq=4, Hkv=2, d=16):
    r = np.random.default_rng(seed)
    V = r.standard_normal((B, L, Hkv, d)).astype(np.float32)
    W = (r.standard_normal((Hq, Hkv * d)) / np.sqrt(Hkv * d)).astype(np.float32)
    A = r.uniform(0.5, 2.0, Hq).astype(np.float32)
    return V, W, A


def test_is_the_linear_layer_over_the_flattened_value_row():
    # the listing's shapes: [b, k_len, n_h * d_h] times the layer's weight [n_h, n_h * d_h] transposed
    V, W, A = _case(1)
    z, dl = oracle.delta_full(V, W, A)
    B, L, Hkv, d = V.shape
    flat = V.astype(np.float64).reshape(B, L, Hkv * d)
    z64 = np.transpose(flat @ W.astype(np.float64).T, (0, 2, 1))
    assert np.allclose(z, z64, rtol=0, atol=1e-5)
    want = np.exp(A.astype(np.float64)[None, :, None] * np.log1p(np.exp(z64)))
    assert np.allclose(dl, want, rtol=2e-6, atol=0)


def test_block_diagonal_weights_give_the_per_head_projection_bit_for_bit():
    # W zero outside the block of head h's own KV head: the extra terms are exact zeros
    V, _, A = _case(2, Hq=6, Hkv=3, d=8)
    r = np.random.default_rng(3)
    Wh = (r.standard_normal((6, 8)) / np.sqrt(8)).astype(np.float32)
    W = np.zeros((6, 3 * 8), np.float32)
    for h in range(6):
        W[h, (h // 2) * 8:(h // 2 + 1) * 8] = Wh[h]
    z_full, dl_full = oracle.delta_full(V, W, A)
    z_head, dl_head = oracle.delta(V, Wh, A, 6)
    assert np.array_equal(z_full.view(np.uint32), z_head.view(np.uint32))
    assert np.array_equal(dl_full.view(np.uint32), dl_head.view(np.uint32))


def test_heads_are_added_left_to_right():
    # three KV heads whose per-head dots are 2^24, 1, -2^24 exactly: ((2^24 + 1) + -2^24) = 0 in fp32, while any
    # other association gives 1
    V = np.zeros((1, 1, 3, 8), np.float32)
    V[0, 0, 0, 0] = 2.0 ** 24; V[0, 0, 1, 0] = 1.0; V[0, 0, 2, 0] = -2.0 ** 24
    W = np.zeros((1, 24), np.float32)
    W[0, 0] = W[0, 8] = W[0, 16] = 1.0
    z, _ = oracle.delta_full(V, W, np.ones(1, np.float32))
    assert z[0, 0, 0] == 0.0
    V[0, 0, 1, 0] = 2.0
    z, _ = oracle.delta_full(V, W, np.ones(1, np.float32))
    assert z[0, 0, 0] == 2.0


def test_one_kv_head_equals_per_head_projection():
    V, W, A = _case(4, Hq=3, Hkv=1, d=32)
    z_full, dl_full = oracle.delta_full(V, W, A)
    z_head, dl_head = oracle.delta(V, W, A, 3)
    assert np.array_equal(z_full, z_head) and np.array_equal(dl_full, dl_head)


def _forward64(V, W, A):
    B, L, Hkv, d = V.shape
    z = np.einsum("blc,hc->bhl", V.reshape(B, L, Hkv * d), W)
    return np.exp(A[None, :, None] * np.log(1.0 + np.exp(z)))


def test_gradient_matches_central_differences():
    V, W, A = (a.astype(np.float64) for a in _case(5, B=2, L=7, Hq=4, Hkv=2, d=8))
    r = np.random.default_rng(6)
    dM = r.standard_normal((2, 4, 7))
    dV, dW, dA = oracle.mask_backward_full(V, W, A, dM)
    loss = lambda V_, W_, A_: float((dM * _forward64(V_, W_, A_)).sum())
    eps = 1e-6
    for _ in range(12):
        idx = tuple(r.integers(0, s) for s in V.shape)
        Vp, Vm = V.copy(), V.copy(); Vp[idx] += eps; Vm[idx] -= eps
        assert abs((loss(Vp, W, A) - loss(Vm, W, A)) / (2 * eps) - dV[idx]) < 1e-5 * max(1.0, abs(dV[idx]))
        idw = tuple(r.integers(0, s) for s in W.shape)
        Wp, Wm = W.copy(), W.copy(); Wp[idw] += eps; Wm[idw] -= eps
        assert abs((loss(V, Wp, A) - loss(V, Wm, A)) / (2 * eps) - dW[idw]) < 1e-5 * max(1.0, abs(dW[idw]))
    for h in range(4):
        Ap, Am = A.copy(), A.copy(); Ap[h] += eps; Am[h] -= eps
        assert abs((loss(V, W, Ap) - loss(V, W, Am)) / (2 * eps) - dA[h]) < 1e-5 * max(1.0, abs(dA[h]))


def test_gradient_reduces_to_the_per_head_one_for_block_diagonal_weights():
    V, _, A = (a.astype(np.float64) for a in _case(7, Hq=4, Hkv=2, d=8))
    r = np.random.default_rng(8)
    Wh = r.standard_normal((4, 8)) / np.sqrt(8)
    W = np.zeros((4, 16))
    for h in range(4):
        W[h, (h // 2) * 8:(h // 2 + 1) * 8] = Wh[h]
    dM = r.standard_normal((2, 4, 11))
    dV, dW, dA = oracle.mask_backward_full(V, W, A, dM)
    dVh, dWh, dAh = oracle.mask_backward(V, Wh, A, dM, 4)
    assert np.allclose(dV, dVh) and np.allclose(dA, dAh)
    for h in range(4):
        assert np.allclose(dW[h, (h // 2) * 8:(h // 2 + 1) * 8], dWh[h])
