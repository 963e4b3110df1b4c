"""ctypes binding of ``libdma_b200.so`` (declared in ``include/dma.h``): argument marshalling only.

Every function here has the name of the C entry point it calls. Tensors are torch CUDA tensors used as
device memory; the current torch stream is passed as the CUDA stream. There is no fallback: if the library is
not built, or a call returns an error status, a ``DmaError`` is raised.
"""
import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdma_b200.so")
_lib = None

DMA_BF16, DMA_FP32 = 0, 1
DMA_FLAG_IGNORE_BITMAP, DMA_FLAG_SIMT, DMA_FLAG_COMPACT_KV, DMA_FLAG_FULL_DELTA, DMA_FLAG_TILE_PATH = 1, 2, 4, 8, 16
DMA_FLAG_BLOCK_SKIP, DMA_FLAG_DETERMINISTIC = 32, 64

ENTRY_POINTS = ("dma_query_workspace", "dma_bitmap_words", "dma_mask_build", "dma_attn_fwd", "dma_attn_bwd",
                "dma_read_status", "dma_launch_count", "dma_strerror", "dma_step_host_arena", "dma_step_host", "dma_mask_build_static", "dma_selftest_wait_timeout",
                "dma_mask_bwd_workspace", "dma_mask_bwd", "dma_delta_range", "dma_decode_workspace", "dma_decode",
                "dma_mask_build_varlen", "dma_decode_state_bytes", "dma_decode_state_init", "dma_decode_step",
                "dma_attn_fwd_chunk", "dma_kernel_timing", "dma_kernel_timing_read")


class DmaError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: status {status} ({dma_strerror(status)})")


class dma_problem_t(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("L", ctypes.c_int32),
                ("d", ctypes.c_int32), ("w", ctypes.c_int32), ("causal", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float),
                ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
                ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3)]


def lib():
    """Loads the shared library; raises if it has not been built (``python -m paper_2508_02124_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise DmaError(-6, f"{LIB_PATH} is missing: build it with `python -m paper_2508_02124_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.dma_strerror.restype = ctypes.c_char_p
        L.dma_launch_count.restype = ctypes.c_longlong
        _lib = L
    return _lib


def dma_strerror(status):
    try:
        return lib().dma_strerror(int(status)).decode()
    except Exception:
        return "?"


def problem(B, Hq, Hkv, L, d, w, dtype=torch.bfloat16, causal=1, tile_m=0, tile_n=0, flags=0, softmax_scale=0.0):
    p = dma_problem_t()
    p.B, p.Hq, p.Hkv, p.L, p.d, p.w, p.causal = B, Hq, Hkv, L, d, w, causal
    if dtype in (torch.bfloat16, torch.float32):
        p.dtype = DMA_BF16 if dtype == torch.bfloat16 else DMA_FP32
    elif type(dtype) is int and dtype in (DMA_BF16, DMA_FP32):
        p.dtype = dtype
    else:
        raise TypeError(f"element type {dtype!r}: torch.bfloat16, torch.float32, DMA_BF16 or DMA_FP32")
    p.tile_m, p.tile_n, p.flags, p.softmax_scale = tile_m, tile_n, flags, softmax_scale
    return p


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _elem(p, *tensors):
    """The library reads Q, K, V, ... as the problem's element type; a tensor of another type would be read out of bounds."""
    want = torch.bfloat16 if p.dtype == DMA_BF16 else torch.float32
    for t in tensors:
        if t is not None and t.dtype != want:
            raise TypeError(f"tensor of {t.dtype} passed for a problem whose element type is {want}")


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, what):
    if rc != 0:
        raise DmaError(rc, what)


def dma_query_workspace(p):
    m, f, b = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().dma_query_workspace(ctypes.byref(p), ctypes.byref(m), ctypes.byref(f), ctypes.byref(b)), "dma_query_workspace")
    return m.value, f.value, b.value


def dma_bitmap_words(p):
    n = ctypes.c_size_t()
    _check(lib().dma_bitmap_words(ctypes.byref(p), ctypes.byref(n)), "dma_bitmap_words")
    return n.value


def _ws(nbytes, device):
    return torch.empty((nbytes + 255) // 256 * 256, dtype=torch.uint8, device=device)


def dma_mask_build(p, V, W_delta, A, bias=None, expiry=None, bitmap=None, ws=None):
    """Returns (bias [B,Hq,L] fp32, expiry [B,Hq,L] int32, bitmap [B,Hq,Tr,ceil(Tc/32)] int32-typed uint32 words)."""
    _elem(p, V)
    dev = V.device
    if bias is None:
        bias = torch.empty(p.B, p.Hq, p.L, dtype=torch.float32, device=dev)
    if expiry is None:
        expiry = torch.empty(p.B, p.Hq, p.L, dtype=torch.int32, device=dev)
    if bitmap is None:
        tm, tn = (p.tile_m or 128), (p.tile_n or 128)
        Tr, Tc = -(-p.L // tm), -(-p.L // tn)
        bitmap = torch.empty(p.B, p.Hq, Tr, (Tc + 31) // 32, dtype=torch.int32, device=dev)
    if ws is None:
        ws = _ws(dma_query_workspace(p)[0], dev)
    _check(lib().dma_mask_build(ctypes.byref(p), _ptr(V), _ptr(W_delta), _ptr(A), _ptr(bias), _ptr(expiry), _ptr(bitmap),
                                _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_mask_build")
    return bias, expiry, bitmap


def dma_mask_build_varlen(p, V, W_delta, A, cu_seqlens, bias=None, expiry=None, bitmap=None, ws=None):
    """dma_mask_build for sequences packed along the sequence axis; cu_seqlens: int32 device tensor [nseq + 1]."""
    _elem(p, V)
    dev = V.device
    assert cu_seqlens.dtype == torch.int32 and cu_seqlens.is_cuda and cu_seqlens.is_contiguous()
    if bias is None:
        bias = torch.empty(p.B, p.Hq, p.L, dtype=torch.float32, device=dev)
    if expiry is None:
        expiry = torch.empty(p.B, p.Hq, p.L, dtype=torch.int32, device=dev)
    if bitmap is None:
        tm, tn = (p.tile_m or 128), (p.tile_n or 128)
        Tr, Tc = -(-p.L // tm), -(-p.L // tn)
        bitmap = torch.empty(p.B, p.Hq, Tr, (Tc + 31) // 32, dtype=torch.int32, device=dev)
    if ws is None:
        ws = _ws(dma_query_workspace(p)[0], dev)
    _check(lib().dma_mask_build_varlen(ctypes.byref(p), _ptr(V), _ptr(W_delta), _ptr(A), _ptr(cu_seqlens),
                                       ctypes.c_int32(cu_seqlens.numel() - 1), _ptr(bias), _ptr(expiry), _ptr(bitmap),
                                       _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_mask_build_varlen")
    return bias, expiry, bitmap


def dma_mask_bwd_workspace(p):
    n = ctypes.c_size_t()
    _check(lib().dma_mask_bwd_workspace(ctypes.byref(p), ctypes.byref(n)), "dma_mask_bwd_workspace")
    return n.value


def dma_mask_bwd(p, V, W_delta, A, bias, dM, dV, dW_delta=None, dA=None, ws=None):
    """Adds the mask path's contribution to dV in place; returns (dV, dW_delta fp32 shaped like W_delta, dA [Hq] fp32)."""
    _elem(p, V, dV)
    dev = V.device
    if dW_delta is None:
        dW_delta = torch.empty(p.Hq, p.Hkv * p.d if p.flags & DMA_FLAG_FULL_DELTA else p.d, dtype=torch.float32, device=dev)
    if dA is None:
        dA = torch.empty(p.Hq, dtype=torch.float32, device=dev)
    if ws is None:
        ws = _ws(dma_mask_bwd_workspace(p), dev)
    _check(lib().dma_mask_bwd(ctypes.byref(p), _ptr(V), _ptr(W_delta), _ptr(A), _ptr(bias), _ptr(dM), _ptr(dV), _ptr(dW_delta),
                              _ptr(dA), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_mask_bwd")
    return dV, dW_delta, dA


def dma_delta_range(p, V, W_delta, A, delta, j_begin, j_end):
    """delta[b,h,j] for the keys j in [j_begin, j_end) of the cache V, written into the delta cache [B,Hq,ld]."""
    _elem(p, V)
    _check(lib().dma_delta_range(ctypes.byref(p), _ptr(V), _ptr(W_delta), _ptr(A), _ptr(delta), ctypes.c_int64(delta.stride(1)),
                                 ctypes.c_int32(j_begin), ctypes.c_int32(j_end), _stream()), "dma_delta_range")
    return delta


def dma_decode_workspace(p):
    n = ctypes.c_size_t()
    _check(lib().dma_decode_workspace(ctypes.byref(p), ctypes.byref(n)), "dma_decode_workspace")
    return n.value


def dma_decode(p, q, K, V, delta, o=None, lse=None, sel_idx=None, want_idx=False, ws=None):
    """One decoding step over the cached keys; returns (o [B,Hq,d], lse [B,Hq], sel_idx or None)."""
    _elem(p, q, K, V, o)
    dev = q.device
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(p.B, p.Hq, dtype=torch.float32, device=dev)
    if sel_idx is None and want_idx:
        sel_idx = torch.empty(p.B, p.Hq, min(p.w, p.L), dtype=torch.int32, device=dev)
    if ws is None:
        ws = _ws(dma_decode_workspace(p), dev)
    _check(lib().dma_decode(ctypes.byref(p), _ptr(q), _ptr(K), _ptr(V), _ptr(delta), ctypes.c_int64(delta.stride(1)), _ptr(o),
                            _ptr(lse), _ptr(sel_idx), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_decode")
    return o, lse, sel_idx


def dma_decode_state(p, device):
    """Zero-filled incremental decoding state for (B, Hq, w): int32 [B*Hq, 8 + roundup(w, 4)] (count 0 everywhere)."""
    n = ctypes.c_size_t()
    _check(lib().dma_decode_state_bytes(ctypes.byref(p), ctypes.byref(n)), "dma_decode_state_bytes")
    return torch.zeros(p.B * p.Hq, n.value // 4 // (p.B * p.Hq), dtype=torch.int32, device=device)


def dma_decode_state_init(p, delta, state, ws=None):
    if ws is None:
        ws = _ws(dma_decode_workspace(p), delta.device)
    _check(lib().dma_decode_state_init(ctypes.byref(p), _ptr(delta), ctypes.c_int64(delta.stride(1)), _ptr(state), _ptr(ws),
                                       ctypes.c_size_t(ws.numel()), _stream()), "dma_decode_state_init")
    return state


def dma_decode_step(p, q, K, V, delta, state, o=None, lse=None, ws=None):
    """One decoding step with the carried state (p.L counts the cached keys including the one just appended)."""
    _elem(p, q, K, V, o)
    dev = q.device
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(p.B, p.Hq, dtype=torch.float32, device=dev)
    if ws is None:
        ws = _ws(dma_decode_workspace(p), dev)
    _check(lib().dma_decode_step(ctypes.byref(p), _ptr(q), _ptr(K), _ptr(V), _ptr(delta), ctypes.c_int64(delta.stride(1)),
                                 _ptr(state), _ptr(o), _ptr(lse), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_decode_step")
    return o, lse


def decode_state_sets(state, w):
    """The kept index sets of a state tensor: list over rows of sorted Python lists."""
    st = state.cpu()
    return [sorted(st[r, 8:8 + int(st[r, 0])].tolist()) for r in range(st.shape[0])]


def dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap, O=None, lse=None, ws=None):
    """Returns (O like Q, lse [B,Hq,L] fp32)."""
    _elem(p, Q, K, V, O)
    if O is None:
        O = torch.empty_like(Q)
    if lse is None:
        lse = torch.empty(p.B, p.Hq, p.L, dtype=torch.float32, device=Q.device)
    if ws is None:
        ws = _ws(dma_query_workspace(p)[1], Q.device)
    _check(lib().dma_attn_fwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(bias), _ptr(expiry), _ptr(bitmap), _ptr(O),
                              _ptr(lse), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_attn_fwd")
    return O, lse


def dma_attn_fwd_chunk(p, q_begin, Q, K, V, bias, expiry, O=None, lse=None, ws=None):
    """Forward for the query rows q_begin .. q_begin + Q.shape[1] - 1 of a sequence of p.L keys; returns (O like Q, lse [B,Hq,q_len])."""
    _elem(p, Q, K, V, O)
    q_len = Q.shape[1]
    if O is None:
        O = torch.empty_like(Q)
    if lse is None:
        lse = torch.empty(p.B, p.Hq, q_len, dtype=torch.float32, device=Q.device)
    if ws is None:
        pc = dma_problem_t.from_buffer_copy(bytes(p))
        pc.flags |= DMA_FLAG_COMPACT_KV
        ws = _ws(dma_query_workspace(pc)[1], Q.device)
    _check(lib().dma_attn_fwd_chunk(ctypes.byref(p), ctypes.c_int32(q_begin), ctypes.c_int32(q_len), _ptr(Q), _ptr(K), _ptr(V),
                                    _ptr(bias), _ptr(expiry), _ptr(O), _ptr(lse), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream()),
           "dma_attn_fwd_chunk")
    return O, lse


def dma_attn_bwd(p, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ=None, dK=None, dV=None, dM=None, ws=None):
    """Returns (dQ like Q, dK like K, dV like V, dM [B,Hq,L] fp32)."""
    _elem(p, Q, K, V, O, dO, dQ, dK, dV)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    if dM is None:
        dM = torch.empty(p.B, p.Hq, p.L, dtype=torch.float32, device=Q.device)
    if ws is None:
        ws = _ws(dma_query_workspace(p)[2], Q.device)
    _check(lib().dma_attn_bwd(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(lse), _ptr(bias),
                              _ptr(expiry), _ptr(bitmap), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dM), _ptr(ws),
                              ctypes.c_size_t(ws.numel()), _stream()), "dma_attn_bwd")
    return dQ, dK, dV, dM


def dma_read_status(ws):
    return lib().dma_read_status(_ptr(ws), _stream())


def dma_launch_count():
    return lib().dma_launch_count()


def dma_kernel_timing(enable):
    """Starts (discarding earlier records) or stops the recording of event pairs around each attention call's main kernel."""
    _check(lib().dma_kernel_timing(int(bool(enable))), "dma_kernel_timing")


def dma_kernel_timing_read(capacity=4096):
    """[(stage, ms), ...] of the launches recorded so far, in call order; stage is "fwd" or "bwd"."""
    ms = (ctypes.c_float * capacity)()
    which = (ctypes.c_int32 * capacity)()
    n = ctypes.c_int32()
    _check(lib().dma_kernel_timing_read(ms, which, capacity, ctypes.byref(n)), "dma_kernel_timing_read")
    return [("bwd" if which[i] else "fwd", float(ms[i])) for i in range(min(n.value, capacity))]


def dma_step_host_arena(p, backward):
    n = ctypes.c_size_t()
    _check(lib().dma_step_host_arena(ctypes.byref(p), int(backward), ctypes.byref(n)), "dma_step_host_arena")
    return n.value


def dma_step_host(p, backward, hQ, hK, hV, hdO, hW, hA, hO, hlse, hdQ, hdK, hdV, hdM, arena):
    """All h* are CPU tensors (ideally pinned); `arena` is a CUDA uint8 tensor of dma_step_host_arena() bytes."""
    _check(lib().dma_step_host(ctypes.byref(p), int(backward), _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(hdO), _ptr(hW), _ptr(hA),
                               _ptr(hO), _ptr(hlse), _ptr(hdQ), _ptr(hdK), _ptr(hdV), _ptr(hdM), _ptr(arena),
                               ctypes.c_size_t(arena.numel()), _stream()), "dma_step_host")


def dma_mask_build_static(p, V, W_delta, A, bias, expiry, bitmap):
    """dma_mask_build without a workspace: the scratch is a fixed array inside the library (see include/dma.h for
    the size limit and the sharing rules). Outputs must be preallocated by the caller; nothing is allocated here."""
    _elem(p, V)
    _check(lib().dma_mask_build_static(ctypes.byref(p), _ptr(V), _ptr(W_delta), _ptr(A), _ptr(bias), _ptr(expiry),
                                       _ptr(bitmap), _stream()), "dma_mask_build_static")
    return bias, expiry, bitmap


def dma_selftest_wait_timeout(ws):
    """Launches the bounded-wait self test; afterwards dma_read_status(ws) reports DMA_ERR_DEVICE_TIMEOUT (-7)."""
    _check(lib().dma_selftest_wait_timeout(_ptr(ws), ctypes.c_size_t(ws.numel()), _stream()), "dma_selftest_wait_timeout")
