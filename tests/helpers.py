"""Shared test plumbing: run a workload through the C-ABI on the GPU, and through the CPU oracle."""
import json
import os

import numpy as np
import torch

import oracle
from paper_2508_02124_b200 import binding as dma

# Parity gate by element type: (max-abs, whole-tensor relative L2). bf16: 2e-2 / 5e-3; fp32: 1e-4 / 1e-4.
# The max-abs bound is read as absolute for tensors of unit scale and as relative to the tensor's largest
# magnitude M beyond that (tol = atol * max(1, M)): half the spacing of bf16, the OUTPUT format, is 2^-8 M, P and dS
# enter the tensor-core GEMMs rounded to bf16, D = rowsum(dO o O) is formed from the stored bf16 O, and dK, dV, dM are
# sums over up to L query rows. The log-sum-exp is an fp32 output whatever the element type: it carries the bias
# magnitude (1e2..1e4) and is held to atol + 1e-6 M, a few fp32 ulps of that magnitude.
TOL = {"bf16": (2e-2, 5e-3), "fp32": (1e-4, 1e-4)}


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


def gpu_run(case, inp, backward=True, mask=None, **kw):
    """Full path on the GPU. `mask` = (bias, expiry, bitmap) CPU/GPU tensors to inject instead of building one."""
    dev = torch.device("cuda:0")
    p = problem_of(case, **kw)
    Q, K, V, dO = (inp[k].to(dev) for k in ("Q", "K", "V", "dO"))
    if mask is None:
        bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(dev), inp["A"].to(dev))
    else:
        bias, expiry, bitmap = (torch.as_tensor(m).to(dev) for m in mask)
    O, lse = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
    out = {"bias": bias, "expiry": expiry, "bitmap": bitmap, "O": O, "lse": lse}
    if backward:
        dQ, dK, dV, dM = dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, bias, expiry, bitmap)
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


def assert_close(got, ref, dtype, what, lse=False):
    g = f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    atol, tol_rel = TOL[dtype]
    diff = np.abs(g - ref)
    M = float(np.abs(ref[np.isfinite(ref)]).max()) if np.isfinite(ref).any() else 0.0
    tol_abs = atol + 1e-6 * M if lse else atol * max(1.0, M)
    den = np.sqrt((ref * ref).sum())
    rel = float(np.sqrt((diff * diff).sum()) / den) if den > 0 else float(diff.max())
    if os.environ.get("DMA_PARITY_LOG"):          # optional record of the measured errors (one JSON line per check)
        with open(os.environ["DMA_PARITY_LOG"], "a") as f:
            f.write(json.dumps({"test": os.environ.get("PYTEST_CURRENT_TEST", ""), "what": what, "dtype": dtype,
                                "max_abs": float(diff.max()), "tol_abs": tol_abs, "rel_l2": rel, "ref_max": M}) + "\n")
    assert np.isfinite(g).all(), f"{what}: non-finite values"
    assert diff.max() <= tol_abs and rel <= tol_rel, (f"{what}: max-abs {diff.max():.3e} (tol {tol_abs:.2e}, |ref| max "
                                                     f"{M:.3e}), rel-L2 {rel:.3e} (tol {tol_rel:.1e})")
    return float(diff.max()), rel
