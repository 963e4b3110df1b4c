"""Seeded synthetic inputs shaped like the paper's kernel workloads (Sec. 5.2, Table "Speed Benchmark
Configurations": 32 query heads, 8 KV heads, head dim 128, bf16).

This module holds input recipes only, none of the method's arithmetic; it is the one module that both
the tests of the CPU oracle and the callers of the CUDA path use. Everything is drawn on the CPU from a
``torch.Generator`` in the fixed order Q, K, V, dO, W_delta, A, positions, in fp32, then rounded to the
case's element type, so that both sides see the same rounded values.
"""
import math
from dataclasses import dataclass, field, replace

import torch


@dataclass(frozen=True)
class Case:
    name: str
    B: int
    Hq: int
    Hkv: int
    L: int
    d: int
    w: int
    dtype: str = "bf16"          # element type of Q,K,V,O,dO,dQ,dK,dV: "bf16" | "fp32"
    backward: bool = True
    seed: int = 0
    qk_scale: float = 1.0        # Q and K multiplied by this (peaked-softmax rerun)
    boost_rows: int = 0          # this many random V rows are scaled x4 (content-driven selection)
    structured: bool = False     # supplementary workload: V built so that V.W_delta follows head archetypes
    causal: int = 1
    extra: dict = field(default_factory=dict)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


# The five benchmark configurations (ids 1..5) plus the supplementary structured workload "S".
CONFIGS = {
    "1": Case("cfg1-tiny-fp32", 1, 2, 2, 256, 64, 64, "fp32", True, 1000),
    "2": Case("cfg2-prefill-4k", 2, 16, 4, 4096, 128, 1024, "bf16", False, 2000),
    "3": Case("cfg3-train-16k", 1, 32, 8, 16384, 128, 2048, "bf16", True, 3000),
    "3x3": Case("cfg3-train-16k-qk3", 1, 32, 8, 16384, 128, 2048, "bf16", True, 3001, qk_scale=3.0),
    "5": Case("cfg5-prefill-64k", 1, 32, 8, 65536, 128, 4096, "bf16", False, 5000, boost_rows=16),
    "S": Case("cfgS-structured-16k", 1, 32, 8, 16384, 128, 2048, "bf16", True, 9000, structured=True),
}
for _i, _w in enumerate((256, 512, 1024, 2048, 4096, 8192)):
    CONFIGS[f"4w{_w}"] = Case(f"cfg4-sweep-8k-w{_w}", 1, 16, 16, 8192, 128, _w, "bf16", True, 4000 + _i)


def small(case: Case, **kw) -> Case:
    """The same recipe at other sizes (parity cases the oracle finishes in seconds)."""
    return replace(case, **kw)


def _structured_z(case: Case, g: torch.Generator) -> torch.Tensor:
    """Target pre-activations z*[Hq, L] for the structured workload, by head archetype (Sec. 6, head
    specialisation: local, long-range, global). Head h takes archetype h % 3. The amplitudes keep delta =
    exp(A softplus(z)) below about 3e3, where fp32 scores still resolve the q.k term."""
    L, Hq = case.L, case.Hq
    pos = torch.arange(L, dtype=torch.float32)
    z = torch.empty(Hq, L)
    for h in range(Hq):
        noise = torch.randn(L, generator=g)
        kind = h % 3
        if kind == 0:        # local: importance grows with position -> sliding band
            z[h] = 3.0 * pos / L + 0.05 * noise
        elif kind == 1:      # long-range: a quarter of the 512-key segments are hot
            nseg = (L + 511) // 512
            hot = (torch.rand(nseg, generator=g) < 0.25).float()
            z[h] = 3.0 * hot.repeat_interleave(512)[:L] + 0.3 * noise
        else:                # global: i.i.d.
            z[h] = noise
    return z


def full_delta_weights(case: Case) -> torch.Tensor:
    """Sampling weights over the whole value row, [Hq, Hkv*d] fp32 ~ N(0, 1/(Hkv*d)) (the z scale of the per-head
    recipe), from the case's seed."""
    g = torch.Generator().manual_seed(case.seed + 77)
    c = case.Hkv * case.d
    return (torch.randn(case.Hq, c, generator=g) / math.sqrt(c)).contiguous()


def packed_cu_seqlens(L: int, nseq: int, seed: int) -> list:
    """Sequence offsets [0, ..., L] of nseq documents packed into L positions: log-normal lengths (a few long
    documents, many short ones, as in packed pre-training batches), every length >= 1, nothing aligned to a tile."""
    g = torch.Generator().manual_seed(seed)
    wts = torch.exp(torch.randn(nseq, generator=g))
    lens = torch.clamp((wts / wts.sum() * (L - nseq)).floor().long() + 1, min=1)
    lens[-1] += L - int(lens.sum())
    assert int(lens.min()) >= 1
    cu = [0]
    for n in lens.tolist():
        cu.append(cu[-1] + n)
    return cu


def make_inputs(case: Case) -> dict:
    """CPU tensors: Q,dO [B,L,Hq,d]; K,V [B,L,Hkv,d] in the case's dtype; W_delta [Hq,d], A [Hq] fp32."""
    g = torch.Generator().manual_seed(case.seed)
    B, L, Hq, Hkv, d = case.B, case.L, case.Hq, case.Hkv, case.d
    Q = torch.randn(B, L, Hq, d, generator=g) * case.qk_scale
    K = torch.randn(B, L, Hkv, d, generator=g) * case.qk_scale
    V = torch.randn(B, L, Hkv, d, generator=g)
    dO = torch.randn(B, L, Hq, d, generator=g)
    W = torch.randn(Hq, d, generator=g) / math.sqrt(d)
    A = torch.rand(Hq, generator=g) * 1.5 + 0.5
    if case.boost_rows:
        pos = torch.randperm(L, generator=g)[: case.boost_rows]
        V[:, pos] *= 4.0
    if case.structured:
        # One KV head feeds G query heads but can follow only one target: use the first head of each group,
        # and give the whole group that head's projection vector so the group shares the pattern.
        G = Hq // Hkv
        zt = _structured_z(case, g)
        for hk in range(Hkv):
            h = hk * G
            W[h: h + G] = W[h]
            wv = W[h]
            cur = V[:, :, hk, :] @ wv                                   # [B, L]
            V[:, :, hk, :] += ((zt[h][None, :] - cur) / wv.dot(wv))[..., None] * wv
    dt = case.torch_dtype
    return {"Q": Q.to(dt), "K": K.to(dt), "V": V.to(dt), "dO": dO.to(dt), "W_delta": W.contiguous(), "A": A}
