"""GPU parity of the incremental decoding step (dma_decode_state_init + dma_decode_step: the kept set carried from step to
step) against the oracle's decoding step evaluated from scratch at every length."""
import numpy as np
import pytest
import torch

import oracle
from paper_2508_02124_b200 import binding as dma
from paper_2508_02124_b200 import workloads as wl
from helpers import assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run(case, n0, steps, seed=5, tie_head=False):
    """The case's K, V form a cache of capacity case.L; the first n0 keys are prefilled (n0 = 0: the sequence starts with
    the first step), then `steps` keys are appended one at a time."""
    inp = wl.make_inputs(case)
    B, cap, Hq, Hkv, d, w = case.B, case.L, case.Hq, case.Hkv, case.d, case.w
    g = torch.Generator().manual_seed(seed)
    A = inp["A"].clone()
    if tie_head:
        A[0] = 0.0                                    # head 0: every delta equals 1, the lowest indices win
    Kd, Vd = inp["K"].to(DEV), inp["V"].to(DEV)
    Wd, Ad = inp["W_delta"].to(DEV), A.to(DEV)
    delta = torch.zeros(B, Hq, cap, device=DEV)
    _, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), A.numpy(), Hq)
    K64, V64 = inp["K"].double().numpy(), inp["V"].double().numpy()

    def problem(n):
        p = dma.problem(B, Hq, Hkv, n, d, w, dtype=case.torch_dtype)
        for s in (p.k_stride, p.v_stride):
            s[0], s[1], s[2] = cap * Hkv * d, Hkv * d, d
        return p

    state = dma.dma_decode_state(problem(max(n0, 1)), DEV)
    if n0 > 0:
        p0 = problem(n0)
        dma.dma_delta_range(p0, Vd, Wd, Ad, delta, 0, n0)
        dma.dma_decode_state_init(p0, delta, state)
    for n in range(n0 + 1, n0 + steps + 1):
        p = problem(n)
        dma.dma_delta_range(p, Vd, Wd, Ad, delta, n - 1, n)
        q = torch.randn(B, Hq, d, generator=g).to(case.torch_dtype)
        o, lse = dma.dma_decode_step(p, q.to(DEV), Kd, Vd, delta, state)
        torch.cuda.synchronize()
        ro, rl, ridx = oracle.decode(q.double().numpy(), K64[:, :n], V64[:, :n], dl[:, :, :n], w)
        sets = dma.decode_state_sets(state, w)
        want = [ridx[b, h].tolist() for b in range(B) for h in range(Hq)]
        assert sets == want, f"kept sets differ at N = {n}"
        assert_close(o, ro, case.dtype, f"{case.name}: o at N = {n}")
        assert_close(lse, rl, case.dtype, f"{case.name}: lse at N = {n}", lse=True)
    return state


@pytest.mark.parametrize("kw,n0,steps", [
    (dict(B=1, Hq=2, Hkv=2, L=64, d=64, w=8, dtype="fp32"), 0, 40),          # from an empty cache through the fill-up
    (dict(B=2, Hq=4, Hkv=2, L=400, d=64, w=100, dtype="bf16"), 90, 60),      # prefill below w: appends, then replacements
    (dict(B=1, Hq=8, Hkv=2, L=1200, d=128, w=300, dtype="bf16"), 1100, 50),  # two list splits, the second ragged
    (dict(B=1, Hq=4, Hkv=4, L=300, d=128, w=1, dtype="fp32"), 200, 40),      # a single kept key
    (dict(B=1, Hq=4, Hkv=1, L=200, d=128, w=4096, dtype="bf16"), 150, 30),   # w above the cache: everything is kept
])
def test_steps_match_the_oracle(kw, n0, steps):
    run(wl.small(wl.CONFIGS["2"], name="decode-step", backward=False, **kw), n0, steps)


def test_ties_go_to_the_lower_index():
    run(wl.small(wl.CONFIGS["2"], B=1, Hq=2, Hkv=1, L=300, d=128, w=50, backward=False, name="decode-step ties"), 40, 80,
        tie_head=True)


def test_state_after_steps_equals_a_fresh_init():
    case = wl.small(wl.CONFIGS["2"], B=1, Hq=4, Hkv=2, L=3000, d=128, w=256, backward=False, name="decode-step vs init")
    state = run(case, 2900, 100)
    inp = wl.make_inputs(case)
    p = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype)
    delta = torch.zeros(case.B, case.Hq, case.L, device=DEV)
    dma.dma_delta_range(p, inp["V"].to(DEV), inp["W_delta"].to(DEV), inp["A"].to(DEV), delta, 0, case.L)
    fresh = dma.dma_decode_state_init(p, delta, dma.dma_decode_state(p, DEV))
    torch.cuda.synchronize()
    assert dma.decode_state_sets(state, case.w) == dma.decode_state_sets(fresh, case.w)
    # the recorded weakest key is the same key in both (its position in the list may differ)
    a, b = state.cpu(), fresh.cpu()
    assert torch.equal(a[:, 2:4], b[:, 2:4])


@pytest.mark.parametrize("seed", range(6))
def test_random_sequences(seed):
    r = np.random.default_rng(40 + seed)
    Hkv, G = int(r.choice([1, 2, 3])), int(r.choice([1, 2, 4]))
    w = int(r.choice([1, 5, 64, 130, 257]))
    n0 = int(r.choice([0, 1, w // 2, w, w + 17, 3 * w]))
    steps = int(r.integers(10, 40))
    case = wl.small(wl.CONFIGS["2"], B=int(r.choice([1, 2])), Hq=Hkv * G, Hkv=Hkv, L=n0 + steps + int(r.integers(0, 9)), d=int(r.choice([64, 128])),
                    w=w, dtype=str(r.choice(["bf16", "fp32"])), backward=False, seed=6000 + seed, name=f"decode-step-random-{seed}")
    run(case, n0, steps, seed=seed, tie_head=bool(seed % 3 == 0))
