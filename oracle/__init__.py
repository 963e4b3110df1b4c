"""CPU oracle for Dynamic Mask Attention: ctypes access to ``dma_oracle.cpp`` (delta in the pinned fp32 arithmetic, the
selection in definition and interval form, bitmaps, forward, backward) plus the parts that are plain numpy in fp64
(mask-generation backward, decoding step, non-causal and packed-sequence selection).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg. The product package never imports it and it never imports the product package.
Arrays are numpy, contiguous, in the layouts documented at the top of ``dma_oracle.cpp``.
"""
import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "dma_oracle.cpp")
_LIB = os.path.join(_DIR, "libdma_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with g++ (no fast-math, no fp contraction: delta-v1 needs exact IEEE ops)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
           _SRC, "-o", _LIB + ".tmp"]
    subprocess.check_call(cmd)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for n in ("dmao_exp_spec", "dmao_log1p_spec", "dmao_softplus_spec"):
            getattr(_lib, n).restype = ctypes.c_float
            getattr(_lib, n).argtypes = [ctypes.c_float]
    return _lib


def threads():
    """Number of OpenMP threads the oracle uses (OMP_NUM_THREADS, else all cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else os.cpu_count()


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


def exp_spec(x):
    return lib().dmao_exp_spec(float(np.float32(x)))


def log1p_spec(t):
    return lib().dmao_log1p_spec(float(np.float32(t)))


def softplus_spec(z):
    return lib().dmao_softplus_spec(float(np.float32(z)))


def delta(V, W, A, Hq):
    """V [B,L,Hkv,d], W [Hq,d], A [Hq] (values exactly representable in fp32) -> (z, delta) [B,Hq,L] fp32."""
    V = _c(V, np.float32); W = _c(W, np.float32); A = _c(A, np.float32)
    B, L, Hkv, d = V.shape
    z = np.empty((B, Hq, L), np.float32)
    dl = np.empty((B, Hq, L), np.float32)
    rc = lib().dmao_delta(_p(V), _p(W), _p(A), B, L, Hq, Hkv, d, _p(z), _p(dl))
    assert rc == 0, rc
    return z, dl


def delta_full(V, W, A):
    """Eq. (delta_calc) with the full sampling weights: V [B,L,Hkv,d], W [Hq, Hkv*d] (one row per query head over the
    flattened value row), A [Hq] -> (z, delta) [B,Hq,L] fp32 in the fixed operation order of the C source."""
    V = _c(V, np.float32); W = _c(W, np.float32); A = _c(A, np.float32)
    B, L, Hkv, d = V.shape
    Hq = W.shape[0]
    assert W.shape == (Hq, Hkv * d) and A.shape == (Hq,)
    z = np.empty((B, Hq, L), np.float32)
    dl = np.empty((B, Hq, L), np.float32)
    rc = lib().dmao_delta_full(_p(V), _p(W), _p(A), B, L, Hq, Hkv, d, _p(z), _p(dl))
    assert rc == 0, rc
    return z, dl


def select_definition(dl, w):
    """delta [..., L] -> keep [..., L, L] uint8 by the per-row sort definition."""
    dl = _c(dl, np.float32)
    L = dl.shape[-1]
    BH = dl.size // L
    keep = np.empty(dl.shape + (L,), np.uint8)
    assert lib().dmao_select_definition(_p(dl), BH, L, int(w), _p(keep)) == 0
    return keep


def select_expiry(dl, w):
    """delta [..., L] -> expiry [..., L] int32: key j is kept by rows j <= i < expiry[j]."""
    dl = _c(dl, np.float32)
    L = dl.shape[-1]
    e = np.empty(dl.shape, np.int32)
    assert lib().dmao_select_expiry(_p(dl), dl.size // L, L, int(w), _p(e)) == 0
    return e


def select_expiry_varlen(dl, w, cu_seqlens):
    """Selection for a batch of sequences packed along the key axis (sequence s owns the keys cu[s] <= j < cu[s+1]):
    every sequence is selected on its own (Sec. 4.1 applied per sequence: a row sees only the keys of its own
    sequence up to itself), so the result is select_expiry of each slice, shifted to packed indices. Key j is then
    kept by the rows j <= i < expiry[j] of the packed axis, and expiry[j] never passes the end of j's sequence."""
    dl = _c(dl, np.float32)
    cu = [int(c) for c in cu_seqlens]
    assert cu[0] == 0 and cu[-1] == dl.shape[-1] and all(a < b for a, b in zip(cu, cu[1:]))
    e = np.empty(dl.shape, np.int32)
    for s0, s1 in zip(cu, cu[1:]):
        e[..., s0:s1] = select_expiry(dl[..., s0:s1], w) + s0
    return e


def select_noncausal(dl, w):
    """Selection without the causal fill (the App. A listing with an all-zero causal_m): every row sees every key, so
    all rows of a head keep the same min(w, L) keys, the best under (delta descending, index ascending). Returned in the
    interval form of the non-causal mode: expiry[j] = L for a kept key, 0 otherwise (key j is kept by rows i < expiry[j])."""
    dl = _c(dl, np.float32)
    L = dl.shape[-1]
    flat = dl.reshape(-1, L)
    e = np.zeros(flat.shape, np.int32)
    pos = np.arange(L)
    for r in range(flat.shape[0]):
        order = np.lexsort((pos, -flat[r].astype(np.float64)))
        e[r, order[:min(int(w), L)]] = L
    return e.reshape(dl.shape)


def keep_from_expiry_noncausal(e):
    e = _c(e, np.int32)
    L = e.shape[-1]
    keep = np.empty(e.shape + (L,), np.uint8)
    assert lib().dmao_keep_from_expiry_noncausal(_p(e), e.size // L, L, _p(keep)) == 0
    return keep


def keep_from_expiry(e):
    e = _c(e, np.int32)
    L = e.shape[-1]
    keep = np.empty(e.shape + (L,), np.uint8)
    assert lib().dmao_keep_from_expiry(_p(e), e.size // L, L, _p(keep)) == 0
    return keep


def _bitmap_shape(lead, L, bm, bn):
    return lead + ((L + bm - 1) // bm, ((L + bn - 1) // bn + 31) // 32)


def bitmap_definition(keep, bm=128, bn=128):
    keep = _c(keep, np.uint8)
    L = keep.shape[-1]
    bmp = np.empty(_bitmap_shape(keep.shape[:-2], L, bm, bn), np.uint32)
    assert lib().dmao_bitmap_definition(_p(keep), keep.size // (L * L), L, bm, bn, _p(bmp)) == 0
    return bmp


def bitmap_from_expiry(e, bm=128, bn=128):
    e = _c(e, np.int32)
    L = e.shape[-1]
    bmp = np.empty(_bitmap_shape(e.shape[:-1], L, bm, bn), np.uint32)
    assert lib().dmao_bitmap_from_expiry(_p(e), e.size // L, L, bm, bn, _p(bmp)) == 0
    return bmp


def forward(Q, K, V, bias, expiry=None, keep=None, scale=None, rows=None, dtype=np.float64, causal=True):
    """Eq. (attention_output). Returns (O, LSE). With ``rows`` only those query rows are evaluated and the
    outputs are compact: O [B,len(rows),Hq,d], LSE [B,Hq,len(rows)]."""
    Q = _c(Q, dtype); K = _c(K, dtype); V = _c(V, dtype); bias = _c(bias, dtype)
    expiry = _c(expiry, np.int32); keep = _c(keep, np.uint8); rows = _c(rows, np.int32)
    B, L, Hq, d = Q.shape
    Hkv = K.shape[2]
    scale = d ** -0.5 if scale is None else scale
    R = L if rows is None else len(rows)
    O = np.empty((B, R, Hq, d), dtype)
    LSE = np.empty((B, Hq, R), dtype)
    f = lib().dmao_fwd_f64 if dtype == np.float64 else lib().dmao_fwd_f32
    rc = f(_p(Q), _p(K), _p(V), _p(bias), _p(expiry), _p(keep), B, L, Hq, Hkv, d, ctypes.c_double(scale),
           _p(rows), 0 if rows is None else len(rows), _p(O), _p(LSE), int(bool(causal)))
    assert rc == 0, rc
    return O, LSE


def backward(Q, K, V, dO, bias, expiry=None, keep=None, scale=None, keys=None, want_dq=True, dtype=np.float64, O=None,
             causal=True):
    """Sec. 4.3 gradients with the mask and bias values held fixed. Returns (dQ, dK, dV, dM). With ``keys`` only
    those keys are evaluated: dK,dV [B,len(keys),Hkv,d], dM [B,Hq,len(keys)] (dQ stays full, or None).
    ``O`` is the stored forward output that Alg. 2 reads for D = rowsum(dO o O); None = the exact output."""
    Q = _c(Q, dtype); K = _c(K, dtype); V = _c(V, dtype); dO = _c(dO, dtype); bias = _c(bias, dtype); O = _c(O, dtype)
    expiry = _c(expiry, np.int32); keep = _c(keep, np.uint8); keys = _c(keys, np.int32)
    B, L, Hq, d = Q.shape
    Hkv = K.shape[2]
    scale = d ** -0.5 if scale is None else scale
    NK = L if keys is None else len(keys)
    dQ = np.empty((B, L, Hq, d), dtype) if want_dq else None
    dK = np.empty((B, NK, Hkv, d), dtype)
    dV = np.empty((B, NK, Hkv, d), dtype)
    dM = np.empty((B, Hq, NK), dtype)
    f = lib().dmao_bwd_f64 if dtype == np.float64 else lib().dmao_bwd_f32
    rc = f(_p(Q), _p(K), _p(V), _p(O), _p(dO), _p(bias), _p(expiry), _p(keep), B, L, Hq, Hkv, d,
           ctypes.c_double(scale), _p(keys), 0 if keys is None else len(keys), _p(dQ), _p(dK), _p(dV), _p(dM),
           int(bool(causal)))
    assert rc == 0, rc
    return dQ, dK, dV, dM


def backward_dq_rows(Q, K, V, dO, bias, rows, expiry=None, keep=None, scale=None, dtype=np.float64, O=None, causal=True):
    """dQ of Sec. 4.3 (Eq. grad_qk) on the listed query rows only (dQ_i depends on row i alone): [B,len(rows),Hq,d].
    ``O`` is the stored forward output of those rows, compact [B,len(rows),Hq,d], that Alg. 2 reads for D; None = the
    exact output."""
    Q = _c(Q, dtype); K = _c(K, dtype); V = _c(V, dtype); dO = _c(dO, dtype); bias = _c(bias, dtype); O = _c(O, dtype)
    expiry = _c(expiry, np.int32); keep = _c(keep, np.uint8); rows = _c(rows, np.int32)
    B, L, Hq, d = Q.shape
    Hkv = K.shape[2]
    scale = d ** -0.5 if scale is None else scale
    assert O is None or O.shape == (B, len(rows), Hq, d)
    dQ = np.empty((B, len(rows), Hq, d), dtype)
    f = lib().dmao_dq_rows_f64 if dtype == np.float64 else lib().dmao_dq_rows_f32
    rc = f(_p(Q), _p(K), _p(V), _p(O), _p(dO), _p(bias), _p(expiry), _p(keep), B, L, Hq, Hkv, d,
           ctypes.c_double(scale), _p(rows), len(rows), _p(dQ), int(bool(causal)))
    assert rc == 0, rc
    return dQ


def mask_backward(V, W, A, dM, Hq):
    """Gradient of the mask-generation bias path (Sec. 4.3: the bias gradient dM reaches the sampling weights and
    the gate; Eq. delta_calc differentiated with the top-w selection held fixed). Plain numpy, fp64:

        z = v . W_h,  sp = softplus(z),  delta = exp(A_h sp)          (forward, per query head h and key j)
        g = dM delta;  dA_h = sum g sp;  dz = g A_h sigmoid(z);  dW_h = sum dz v;  dV[j, kv head] = sum_h dz W_h

    V [B,L,Hkv,d], W [Hq,d], A [Hq], dM [B,Hq,L] -> (dV [B,L,Hkv,d], dW [Hq,d], dA [Hq]); query head h reads KV
    head h // (Hq // Hkv)."""
    V = np.asarray(V, np.float64); W = np.asarray(W, np.float64); A = np.asarray(A, np.float64)
    dM = np.asarray(dM, np.float64)
    B, L, Hkv, d = V.shape
    G = Hq // Hkv
    dV = np.zeros_like(V); dW = np.zeros_like(W); dA = np.zeros_like(A)
    for h in range(Hq):
        hk = h // G
        v = V[:, :, hk, :]                                   # [B, L, d]
        z = v @ W[h]                                         # [B, L]
        sp = np.maximum(z, 0.0) + np.log1p(np.exp(-np.abs(z)))
        delta = np.exp(A[h] * sp)
        g = dM[:, h, :] * delta
        dA[h] = (g * sp).sum()
        sig = np.where(z >= 0, 1.0 / (1.0 + np.exp(-np.abs(z))), np.exp(-np.abs(z)) / (1.0 + np.exp(-np.abs(z))))
        dz = g * A[h] * sig
        dW[h] = np.einsum("bl,bld->d", dz, v)
        dV[:, :, hk, :] += dz[..., None] * W[h]
    return dV, dW, dA


def mask_backward_full(V, W, A, dM):
    """mask_backward for the full sampling weights W [Hq, Hkv*d] (every query head reads the whole value row):

        z = vrow . W_h  (vrow = the Hkv*d channels of key j),  g = dM delta,  dA_h = sum g softplus(z),
        dz = g A_h sigmoid(z),  dW_h = sum dz vrow,  dVrow[j] = sum_h dz W_h

    Plain numpy, fp64. V [B,L,Hkv,d], A [Hq], dM [B,Hq,L] -> (dV like V, dW like W, dA [Hq])."""
    V = np.asarray(V, np.float64); W = np.asarray(W, np.float64); A = np.asarray(A, np.float64)
    dM = np.asarray(dM, np.float64)
    B, L, Hkv, d = V.shape
    rows = V.reshape(B, L, Hkv * d)
    dRows = np.zeros_like(rows); dW = np.zeros_like(W); dA = np.zeros_like(A)
    for h in range(W.shape[0]):
        z = rows @ W[h]                                      # [B, L]
        e = np.exp(-np.abs(z))
        sp = np.maximum(z, 0.0) + np.log1p(e)
        g = dM[:, h, :] * np.exp(A[h] * sp)
        dA[h] = (g * sp).sum()
        dz = g * A[h] * np.where(z >= 0, 1.0, e) / (1.0 + e)
        dW[h] = np.einsum("bl,blc->c", dz, rows)
        dRows += dz[..., None] * W[h]
    return dRows.reshape(V.shape), dW, dA


def decode(q, K, V, delta, w, scale=None):
    """One decoding step (Sec. 3.2 with a single query at the end of the sequence; Alg. 1 with the per-key mask
    M in R^N): the query of every (batch, head) sees all N cached keys, keeps the w with the largest dynamic weight
    delta (ties to the lower index; all of them if N <= w) and attends to those with delta as the additive bias.
    Plain numpy, fp64. q [B,Hq,d], K, V [B,N,Hkv,d], delta [B,Hq,N] (compared as given) ->
    (o [B,Hq,d], lse [B,Hq], idx [B,Hq,min(w,N)] int32 ascending)."""
    q = np.asarray(q, np.float64); K = np.asarray(K, np.float64); V = np.asarray(V, np.float64)
    B, Hq, d = q.shape
    N, Hkv = K.shape[1], K.shape[2]
    G = Hq // Hkv
    scale = d ** -0.5 if scale is None else scale
    keep = min(w, N)
    o = np.empty((B, Hq, d)); lse = np.empty((B, Hq)); idx = np.empty((B, Hq, keep), np.int32)
    pos = np.arange(N)
    for b in range(B):
        for h in range(Hq):
            dl = np.asarray(delta[b, h])
            order = np.lexsort((pos, -dl.astype(np.float64)))[:keep]          # delta descending, then index ascending
            sel = np.sort(order)
            s = (K[b, sel, h // G, :] @ q[b, h]) * scale + dl[sel].astype(np.float64)
            m = s.max()
            p = np.exp(s - m)
            o[b, h] = (p / p.sum()) @ V[b, sel, h // G, :]
            lse[b, h] = m + np.log(p.sum())
            idx[b, h] = sel
    return o, lse, idx
