"""Pins for the oracle's mask-generation backward (Sec. 4.3 / Eq. delta_calc differentiated): central finite
differences of an independently written forward, closed forms, linearity and the GQA group sum."""
import numpy as np

import oracle


def _delta_forward(V, W, A, Hq):
    """delta = exp(A softplus(V.W)) written directly from Eq. delta_calc (fp64, naive softplus is fine at these sizes)."""
    B, L, Hkv, d = V.shape
    G = Hq // Hkv
    out = np.empty((B, Hq, L))
    for h in range(Hq):
        z = V[:, :, h // G, :] @ W[h]
        out[:, h, :] = np.exp(A[h] * np.log(1.0 + np.exp(z)))
    return out


def _case(seed, B=2, L=9, Hq=4, Hkv=2, d=8):
    r = np.random.default_rng(seed)
    return (r.standard_normal((B, L, Hkv, d)), r.standard_normal((Hq, d)) / np.sqrt(d), r.uniform(0.5, 2.0, Hq),
            r.standard_normal((B, Hq, L)), Hq)


def test_matches_central_differences():
    V, W, A, dM, Hq = _case(1)
    dV, dW, dA = oracle.mask_backward(V, W, A, dM, Hq)
    loss = lambda V_, W_, A_: float((dM * _delta_forward(V_, W_, A_, Hq)).sum())
    eps = 1e-6
    r = np.random.default_rng(2)
    for _ in range(12):
        idx = tuple(r.integers(0, s) for s in V.shape)
        Vp, Vm = V.copy(), V.copy(); Vp[idx] += eps; Vm[idx] -= eps
        assert abs((loss(Vp, W, A) - loss(Vm, W, A)) / (2 * eps) - dV[idx]) < 1e-5 * max(1.0, abs(dV[idx]))
        idw = tuple(r.integers(0, s) for s in W.shape)
        Wp, Wm = W.copy(), W.copy(); Wp[idw] += eps; Wm[idw] -= eps
        assert abs((loss(V, Wp, A) - loss(V, Wm, A)) / (2 * eps) - dW[idw]) < 1e-5 * max(1.0, abs(dW[idw]))
    for h in range(Hq):
        Ap, Am = A.copy(), A.copy(); Ap[h] += eps; Am[h] -= eps
        assert abs((loss(V, W, Ap) - loss(V, W, Am)) / (2 * eps) - dA[h]) < 1e-5 * max(1.0, abs(dA[h]))


def test_zero_values_closed_form():
    # V = 0: z = 0, softplus = ln 2, delta = 2^A, sigmoid = 1/2
    _, W, A, dM, Hq = _case(3)
    V = np.zeros((2, 9, 2, 8))
    dV, dW, dA = oracle.mask_backward(V, W, A, dM, Hq)
    assert np.allclose(dW, 0.0)
    assert np.allclose(dA, dM.sum(axis=(0, 2)) * 2.0 ** A * np.log(2.0))
    coef = dM * (2.0 ** A * A * 0.5)[None, :, None]                      # dz [B, Hq, L]
    want = np.zeros_like(V)
    for h in range(Hq):
        want[:, :, h // 2, :] += coef[:, h, :, None] * W[h]
    assert np.allclose(dV, want)


def test_zero_gate_only_dA_survives():
    # A = 0: delta = 1 whatever z is, so dz = 0; dA = sum dM softplus(z)
    V, W, _, dM, Hq = _case(4)
    A = np.zeros(Hq)
    dV, dW, dA = oracle.mask_backward(V, W, A, dM, Hq)
    assert np.allclose(dV, 0.0) and np.allclose(dW, 0.0)
    sp = np.stack([np.log1p(np.exp(V[:, :, h // 2, :] @ W[h])) for h in range(Hq)], axis=1)
    assert np.allclose(dA, (dM * sp).sum(axis=(0, 2)))


def test_linear_in_dM_and_large_z_is_stable():
    V, W, A, dM, Hq = _case(5)
    a = oracle.mask_backward(V, W, A, dM, Hq)
    b = oracle.mask_backward(V, W, A, 3.0 * dM, Hq)
    for x, y in zip(a, b):
        assert np.allclose(3.0 * x, y)
    big = oracle.mask_backward(40.0 * V, W, 0.01 * A, dM, Hq)            # |z| up to ~100: no overflow in softplus / sigmoid
    assert all(np.isfinite(t).all() for t in big)


def test_group_sum_over_query_heads():
    # a KV head's dV is the sum of what each of its query heads contributes alone
    V, W, A, dM, Hq = _case(6)
    full = oracle.mask_backward(V, W, A, dM, Hq)[0]
    acc = np.zeros_like(full)
    for h in range(Hq):
        one = np.zeros_like(dM); one[:, h, :] = dM[:, h, :]
        acc += oracle.mask_backward(V, W, A, one, Hq)[0]
    assert np.allclose(full, acc)
