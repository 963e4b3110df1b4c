"""Pins for the oracle's forward (Sec. 4.2) and backward (Sec. 4.3): textbook special cases evaluated
with torch library routines, closed forms, invariants and central finite differences."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle


def rand_case(seed, B=2, L=48, Hq=4, Hkv=2, d=16, w=9, ties=False):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, L, Hq, d))
    K = rng.standard_normal((B, L, Hkv, d))
    V = rng.standard_normal((B, L, Hkv, d))
    dO = rng.standard_normal((B, L, Hq, d))
    dl = rng.uniform(1, 4, (B, Hq, L)).astype(np.float32)
    if ties:
        dl = np.round(dl, 0)
    e = oracle.select_expiry(dl, w)
    return Q, K, V, dO, dl.astype(np.float64), e


def torch_masked_attention(Q, K, V, bias, keep, scale=None):
    """Library statement of Eq. (attention_output): SDPA with an additive mask that is bias where kept and
    -inf elsewhere; KV heads repeated over their query-head group. All [B,L,H,d] float64 torch tensors."""
    B, L, Hq, d = Q.shape
    G = Hq // K.shape[2]
    q = Q.permute(0, 2, 1, 3)
    k = K.repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    v = V.repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    add = torch.where(keep.bool(), bias[:, :, None, :].expand(-1, -1, L, -1), torch.tensor(-float("inf"), dtype=Q.dtype))
    s = q @ k.transpose(-1, -2) * (scale if scale is not None else d ** -0.5) + add
    p = torch.softmax(s, dim=-1)
    return (p @ v).permute(0, 2, 1, 3), torch.logsumexp(s, dim=-1)


T = lambda a: torch.tensor(a, dtype=torch.float64)


# ----------------------------------------------------------------------------------------- forward

def test_forward_dense_causal_limit_matches_sdpa():
    # w >= L and a constant bias: exactly dense causal softmax attention (library SDPA, is_causal=True)
    Q, K, V, _, _, _ = rand_case(1, L=40, w=40)
    B, L, Hq, d = Q.shape
    e = np.full((B, Hq, L), L, np.int32)
    for const in (0.0, 3.5):
        O, lse = oracle.forward(Q, K, V, np.full((B, Hq, L), const), expiry=e)
        G = Hq // K.shape[2]
        ref = F.scaled_dot_product_attention(T(Q).permute(0, 2, 1, 3), T(K).repeat_interleave(G, 2).permute(0, 2, 1, 3),
                                             T(V).repeat_interleave(G, 2).permute(0, 2, 1, 3), is_causal=True)
        assert np.abs(O - ref.permute(0, 2, 1, 3).numpy()).max() < 1e-12


def test_forward_sliding_window_limit():
    # increasing delta selects the w latest keys; with zero bias that is textbook sliding-window attention
    Q, K, V, _, _, _ = rand_case(2, L=50, w=7)
    B, L, Hq, d = Q.shape
    w = 7
    e = oracle.select_expiry(np.broadcast_to(np.linspace(1, 2, L, dtype=np.float32), (B, Hq, L)), w)
    O, lse = oracle.forward(Q, K, V, np.zeros((B, Hq, L)), expiry=e)
    i = torch.arange(L)
    band = (i[None, :] <= i[:, None]) & (i[None, :] > i[:, None] - w)
    ref, ref_lse = torch_masked_attention(T(Q), T(K), T(V), torch.zeros(B, Hq, L, dtype=torch.float64), band[None, None].expand(B, Hq, -1, -1))
    assert np.abs(O - ref.numpy()).max() < 1e-12 and np.abs(lse - ref_lse.numpy()).max() < 1e-12


@pytest.mark.parametrize("ties", [False, True])
def test_forward_general_mask_matches_library_softmax(ties):
    Q, K, V, _, bias, e = rand_case(3, ties=ties)
    keep = oracle.keep_from_expiry(e)
    ref, ref_lse = torch_masked_attention(T(Q), T(K), T(V), T(bias), torch.tensor(keep))
    for kw in (dict(expiry=e), dict(keep=keep)):
        O, lse = oracle.forward(Q, K, V, bias, **kw)
        assert np.abs(O - ref.numpy()).max() < 1e-11 and np.abs(lse - ref_lse.numpy()).max() < 1e-11
    # custom scale, and the fp32 instantiation agrees to fp32 accuracy
    O, _ = oracle.forward(Q, K, V, bias, expiry=e, scale=0.3)
    ref, _ = torch_masked_attention(T(Q), T(K), T(V), T(bias), torch.tensor(keep), scale=0.3)
    assert np.abs(O - ref.numpy()).max() < 1e-11
    O32, lse32 = oracle.forward(Q, K, V, bias, expiry=e, scale=0.3, dtype=np.float32)
    assert np.abs(O32 - ref.numpy()).max() < 2e-5


def test_forward_invariants_and_closed_forms():
    Q, K, V, _, bias, e = rand_case(4, B=1, L=64, w=11)
    B, L, Hq, d = Q.shape
    G = Hq // K.shape[2]
    O, lse = oracle.forward(Q, K, V, bias, expiry=e)
    # rows of P sum to one: constant values come back unchanged
    O1, _ = oracle.forward(Q, K, np.ones_like(V), bias, expiry=e)
    assert np.abs(O1 - 1).max() < 1e-13
    # shifting the bias by a constant leaves O and moves LSE by that constant
    O2, lse2 = oracle.forward(Q, K, V, bias + 2.25, expiry=e)
    assert np.abs(O2 - O).max() < 1e-12 and np.abs(lse2 - lse - 2.25).max() < 1e-12
    # Q = 0: the weights are softmax of the kept biases alone
    O3, _ = oracle.forward(np.zeros_like(Q), K, V, bias, expiry=e)
    keep = oracle.keep_from_expiry(e)
    for h in range(Hq):
        for i in (0, 5, 63):
            idx = np.nonzero(keep[0, h, i])[0]
            p = np.exp(bias[0, h, idx] - bias[0, h, idx].max())
            p /= p.sum()
            assert np.abs(O3[0, i, h] - p @ V[0, idx, h // G]).max() < 1e-12
    # w = 1: each row copies the value of its single kept key, and LSE is that key's score
    e1 = oracle.select_expiry(bias.astype(np.float32), 1)
    O4, lse4 = oracle.forward(Q, K, V, bias, expiry=e1)
    for h in range(Hq):
        for i in range(L):
            j = int(np.argmax(bias[0, h, : i + 1]))
            assert np.abs(O4[0, i, h] - V[0, j, h // G]).max() < 1e-13
            assert abs(lse4[0, h, i] - (Q[0, i, h] @ K[0, j, h // G] / math.sqrt(d) + bias[0, h, j])) < 1e-12
    # the first row (L = 1 case) sees only key 0
    assert np.abs(O[:, 0] - np.repeat(V[:, 0], G, axis=1)).max() < 1e-13


def test_forward_row_subset_equals_full():
    Q, K, V, _, bias, e = rand_case(5)
    O, lse = oracle.forward(Q, K, V, bias, expiry=e)
    rows = np.array([0, 7, 20, 47], np.int32)
    Os, lses = oracle.forward(Q, K, V, bias, expiry=e, rows=rows)
    assert (Os == O[:, rows]).all() and (lses == lse[:, :, rows]).all()


# ---------------------------------------------------------------------------------------- backward

def loss_terms(Q, K, V, dO, bias, e):
    O, _ = oracle.forward(Q, K, V, bias, expiry=e)
    return float((O * dO).sum())


def test_backward_central_finite_differences():
    # mask (expiry) and bias values are held fixed: the hot path's gradients stop at dM (Eq. grad_m)
    Q, K, V, dO, bias, e = rand_case(6, B=1, L=24, Hq=4, Hkv=2, d=8, w=5)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias, expiry=e)
    rng = np.random.default_rng(0)
    h = 1e-6
    for name, X, grad in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV), ("bias", bias, dM)):
        for _ in range(25):
            idx = tuple(rng.integers(0, s) for s in X.shape)
            args = {"Q": Q, "K": K, "V": V, "bias": bias}
            xp, xm = X.copy(), X.copy()
            xp[idx] += h
            xm[idx] -= h
            fp = loss_terms(**{**args, name: xp}, dO=dO, e=e)
            fm = loss_terms(**{**args, name: xm}, dO=dO, e=e)
            fd = (fp - fm) / (2 * h)
            assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


@pytest.mark.parametrize("ties", [False, True])
def test_backward_matches_library_autograd(ties):
    Q, K, V, dO, bias, e = rand_case(7, ties=ties)
    keep = torch.tensor(oracle.keep_from_expiry(e))
    tq, tk, tv, tb = (T(x).requires_grad_() for x in (Q, K, V, bias))
    O, _ = torch_masked_attention(tq, tk, tv, tb, keep)
    O.backward(T(dO))
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias, expiry=e)
    for got, ref in ((dQ, tq.grad), (dK, tk.grad), (dV, tv.grad), (dM, tb.grad)):
        assert np.abs(got - ref.numpy()).max() < 1e-10
    dQ2, dK2, dV2, dM2 = oracle.backward(Q, K, V, dO, bias, keep=keep.numpy())
    assert np.abs(dQ2 - dQ).max() == 0 and np.abs(dK2 - dK).max() == 0 and np.abs(dM2 - dM).max() == 0
    g32 = oracle.backward(Q, K, V, dO, bias, expiry=e, dtype=np.float32)
    for got, ref in zip(g32, (dQ, dK, dV, dM)):
        assert np.abs(got - ref).max() < 5e-5


def test_backward_dense_causal_limit_matches_sdpa_autograd():
    Q, K, V, dO, _, _ = rand_case(8, L=32, w=32)
    B, L, Hq, d = Q.shape
    G = Hq // K.shape[2]
    tq, tk, tv = (T(x).requires_grad_() for x in (Q, K, V))
    ref = F.scaled_dot_product_attention(tq.permute(0, 2, 1, 3), tk.repeat_interleave(G, 2).permute(0, 2, 1, 3),
                                         tv.repeat_interleave(G, 2).permute(0, 2, 1, 3), is_causal=True)
    ref.backward(T(dO).permute(0, 2, 1, 3))
    e = np.full((B, Hq, L), L, np.int32)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, np.zeros((B, Hq, L)), expiry=e)
    assert np.abs(dQ - tq.grad.numpy()).max() < 1e-11
    assert np.abs(dK - tk.grad.numpy()).max() < 1e-11
    assert np.abs(dV - tv.grad.numpy()).max() < 1e-11


def test_backward_invariants():
    Q, K, V, dO, bias, e = rand_case(9, B=2, L=64, Hq=4, Hkv=2, d=16, w=13)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias, expiry=e)
    # each row of dS sums to zero (softmax Jacobian), so dM sums to zero over keys
    assert np.abs(dM.sum(-1)).max() < 1e-11
    # sum_i q_i . dQ_i = sum_j k_j . dK_j  within each KV group (both equal sum_ij dS_ij q_i.k_j scale)
    G = Q.shape[2] // K.shape[2]
    lhs = (Q * dQ).sum(-1).reshape(2, 64, K.shape[2], G).sum((1, 3))
    rhs = (K * dK).sum(-1).sum(1)
    assert np.abs(lhs - rhs).max() < 1e-10
    # w = 1: one kept key per row -> p = 1, dS = 0: no gradient to Q, K or the bias; dV_j collects dO of its rows
    e1 = oracle.select_expiry(bias.astype(np.float32), 1)
    dQ1, dK1, dV1, dM1 = oracle.backward(Q, K, V, dO, bias, expiry=e1)
    assert np.abs(dQ1).max() < 1e-12 and np.abs(dK1).max() < 1e-12 and np.abs(dM1).max() < 1e-12
    ref = np.zeros_like(V)
    for b in range(2):
        for h in range(4):
            for i in range(64):
                ref[b, int(np.argmax(bias[b, h, : i + 1])), h // G] += dO[b, i, h]
    assert np.abs(dV1 - ref).max() < 1e-12


def test_backward_key_subset_equals_full():
    Q, K, V, dO, bias, e = rand_case(10)
    dQ, dK, dV, dM = oracle.backward(Q, K, V, dO, bias, expiry=e)
    keys = np.array([0, 3, 30, 47], np.int32)
    dQs, dKs, dVs, dMs = oracle.backward(Q, K, V, dO, bias, expiry=e, keys=keys, want_dq=False)
    assert dQs is None
    assert (dKs == dK[:, keys]).all() and (dVs == dV[:, keys]).all() and (dMs == dM[:, :, keys]).all()


def test_backward_dq_row_subset_equals_full():
    # dQ_i depends on row i alone: the row-subset routine must reproduce the rows of the full backward (itself pinned by
    # finite differences above), with the exact O and with a stored (here: perturbed) O
    Q, K, V, dO, bias, e = rand_case(12)
    rows = np.array([0, 1, 17, 40, Q.shape[1] - 1], np.int32)
    dQ = oracle.backward(Q, K, V, dO, bias, expiry=e)[0]
    assert (oracle.backward_dq_rows(Q, K, V, dO, bias, rows, expiry=e) == dQ[:, rows]).all()
    O, _ = oracle.forward(Q, K, V, bias, expiry=e)
    O2 = O + 0.01 * np.cos(np.arange(O.size)).reshape(O.shape)
    dQ2 = oracle.backward(Q, K, V, dO, bias, expiry=e, O=O2)[0]
    got = oracle.backward_dq_rows(Q, K, V, dO, bias, rows, expiry=e, O=O2[:, rows])
    assert (got == dQ2[:, rows]).all() and np.abs(dQ2 - dQ).max() > 1e-6
    # definition form (keep matrix) and non-causal mode go through the same routine
    keep = oracle.keep_from_expiry(e)
    assert (oracle.backward_dq_rows(Q, K, V, dO, bias, rows, keep=keep) == dQ[:, rows]).all()


def test_backward_with_stored_output():
    # Alg. 2 reads O back from memory for D = rowsum(dO o O): passing the exact O changes nothing; passing a
    # perturbed O moves D by dO.(O' - O) and hence dS by -p * that, which for dM (column sums of dS) is checkable.
    Q, K, V, dO, bias, e = rand_case(11, B=1, L=40, Hq=2, Hkv=1, d=8, w=6)
    O, _ = oracle.forward(Q, K, V, bias, expiry=e)
    base = oracle.backward(Q, K, V, dO, bias, expiry=e)
    same = oracle.backward(Q, K, V, dO, bias, expiry=e, O=O)
    for a, b in zip(base, same):
        assert np.abs(a - b).max() < 1e-13
    O2 = O + 0.01
    pert = oracle.backward(Q, K, V, dO, bias, expiry=e, O=O2)
    shift = (dO * (O2 - O)).sum(-1)                                    # [B, L, Hq] change of D_i
    keep = oracle.keep_from_expiry(e).astype(np.float64)
    s = np.einsum("blhc,bmhc->bhlm", Q, np.repeat(K, 2, axis=2)) / math.sqrt(8) + bias[:, :, None, :]
    s = np.where(keep > 0, s, -np.inf)
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    expect_dM = base[3] - np.einsum("bhlm,blh->bhm", p, shift)
    assert np.abs(pert[3] - expect_dM).max() < 1e-12
    assert np.abs(pert[2] - base[2]).max() < 1e-13                     # dV does not depend on D
