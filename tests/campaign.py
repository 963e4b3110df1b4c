"""Long randomised campaigns on a GPU, outside the test suite (pytest does not collect this file):

    python tests/campaign.py <name> [seconds] [first seed]

    attention  tensor-core kernels (tile path, token-compacted) against the CUDA-core kernels: causal / packed / non-causal
    mask       dma_mask_build (+ varlen, non-causal, full projection) bit for bit against the oracle, with tie-heavy inputs
    decode     dma_decode_step sequences and dma_decode calls against the oracle at every length
    chunk      dma_attn_fwd_chunk against the rows of the whole-sequence forward
    maskbwd    dma_mask_bwd (per-head and full projection) against the oracle
    strided    strided placements of Q, K, V, O against the packed run of the same path
    host       dma_step_host against the device entry points
    large      ragged lengths up to 65 537: masks bit for bit, tile against compacted path, sampled rows / keys against the oracle

Every case is drawn from numpy's default_rng(seed); a failure prints the seed and the shape. The exit code is the number of
failures (capped at 255)."""
import os
import sys
import time

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))
sys.path.insert(0, HERE)

import oracle  # noqa: E402
from paper_2508_02124_b200 import binding as dma  # noqa: E402
from paper_2508_02124_b200 import workloads as wl  # noqa: E402

DEV = "cuda:0"
TILE = dma.DMA_FLAG_TILE_PATH          # the tile-walking kernels; 0 leaves the choice to the library
C2 = wl.CONFIGS["2"]


class Tally:
    def __init__(self, name, seconds, seed):
        self.name, self.t0, self.budget, self.seed, self.n, self.fails = name, time.time(), seconds, seed, 0, 0

    def running(self):
        return time.time() - self.t0 < self.budget

    def next_rng(self):
        self.seed += 1
        return np.random.default_rng(self.seed)

    def fail(self, *what):
        self.fails += 1
        print("FAIL", self.name, self.seed, *what, flush=True)

    def done(self):
        print(f"{self.name}: {self.n} cases, {self.fails} failures, {time.time() - self.t0:.0f} s, last seed {self.seed}")
        return self.fails


def close(a, b, rel):
    """max-abs difference within rel * max(1, max |b|), and a finite"""
    a, b = a.float(), b.float()
    return bool(torch.isfinite(a).all()) and float((a - b).abs().max()) <= rel * max(1.0, float(b.abs().max()))


def placed(inp, B, L, Hq, Hkv, d, off):
    """Q, K, V, dO as views of one bf16 buffer starting `off` elements in (memory placement changes kernel timing)"""
    nq, nk = B * L * Hq * d, B * L * Hkv * d
    big = torch.empty(2 * nq + 2 * nk + off + 64, dtype=torch.bfloat16, device=DEV)
    o, views = off, {}
    for k, n, H in (("Q", nq, Hq), ("K", nk, Hkv), ("V", nk, Hkv), ("dO", nq, Hq)):
        views[k] = big[o:o + n].view(B, L, H, d)
        views[k].copy_(inp[k])
        o += n
    return views


def run_all_paths(p_of, Q, K, V, dO, mask, order):
    outs = []
    for flags in order:
        p = p_of(flags)
        O, lse = dma.dma_attn_fwd(p, Q, K, V, *mask)
        g = dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, *mask)
        torch.cuda.synchronize()
        outs.append(dict(zip(("O", "lse", "dQ", "dK", "dV", "dM"), (O, lse) + tuple(g))))
    return outs


def attention(T):
    """dM is compared with every path given the CUDA-core path's O: Alg. 2 forms D from the stored, bf16-rounded O, and for
    keys that many rows attend to almost alone dM carries that rounding at full weight."""
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 4, 8])), int(r.choice([1, 2, 4, 8]))
        if Hkv * G > 16:
            G = 16 // Hkv
        L = int(r.choice([130, 257, 384, 777, 1024, 1500, 2048, 3333, 4096, 6000]))
        w = int(r.choice([1, 2, 31, 64, 128, 129, 500, 1024, 2048, 5000]))
        d, B = int(r.choice([64, 128, 128])), int(r.choice([1, 1, 2, 3]))
        causal = int(r.random() < 0.8)
        varlen = bool(causal and r.random() < 0.5)
        cu = [0] + sorted(set(int(c) for c in r.integers(1, L, int(r.integers(2, 16)) - 1))) + [L]
        case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, backward=True, seed=T.seed, name="campaign")
        inp = wl.make_inputs(case)
        v = placed(inp, B, L, case.Hq, Hkv, d, int(r.integers(0, 64)) * 0x2468)
        W, A = inp["W_delta"].to(DEV), inp["A"].to(DEV)
        if not causal:
            A = A * 0.25              # one key set per head: with the causal recipe's gates every row would be one-hot
        p_of = lambda flags: dma.problem(B, case.Hq, Hkv, L, d, w, flags=flags if causal else flags & ~TILE, causal=causal)
        if varlen:
            mask = dma.dma_mask_build_varlen(p_of(0), v["V"], W, A, torch.tensor(cu, dtype=torch.int32, device=DEV))
        else:
            mask = dma.dma_mask_build(p_of(0), v["V"], W, A)
        ref = None
        for flags in (dma.DMA_FLAG_SIMT, TILE, dma.DMA_FLAG_COMPACT_KV, TILE, dma.DMA_FLAG_COMPACT_KV, 0):
            p = p_of(flags)
            O, lse = dma.dma_attn_fwd(p, v["Q"], v["K"], v["V"], *mask)
            g = dma.dma_attn_bwd(p, v["Q"], v["K"], v["V"], ref["O"] if ref else O, v["dO"], ref["lse"] if ref else lse, *mask)
            torch.cuda.synchronize()
            out = dict(zip(("O", "lse", "dQ", "dK", "dV", "dM"), (O, lse) + tuple(g)))
            if ref is None:
                ref = out
                continue
            bad = [k for k, t in out.items() if not close(t, ref[k], 1e-3 if k == "lse" else 4e-2)]
            if bad:
                T.fail(dict(B=B, Hq=case.Hq, Hkv=Hkv, L=L, w=w, d=d, causal=causal, cu=cu if varlen else None), "flags", flags, bad)
        T.n += 1


def mask(T):
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 4])), int(r.choice([1, 2, 4]))
        L = int(r.choice([1, 2, 127, 128, 129, 255, 256, 257, 500, 1000, 1024, 2049, 4096, 5000, 9000]))
        w = int(r.choice([1, 2, 3, 31, 32, 33, 100, 255, 256, 257, 700, 1024, 3000, 10000]))
        d, B = int(r.choice([64, 128])), int(r.choice([1, 2]))
        mode = int(r.integers(0, 4))                      # 0 causal, 1 packed, 2 non-causal, 3 full projection (causal)
        ties = int(r.integers(0, 4))                      # 0 none, 1 quantised V and W, 2 an A = 0 head, 3 a run of equal value rows
        dt = torch.bfloat16 if r.random() < 0.7 else torch.float32
        g = torch.Generator().manual_seed(T.seed)
        Hq = Hkv * G
        V = torch.randn(B, L, Hkv, d, generator=g)
        if ties == 1:
            V = (V * 2).round() / 2
        if ties == 3 and L > 8:
            V[:, L // 3: L // 3 + max(2, L // 4)] = V[:, L // 3: L // 3 + 1]
        V = V.to(dt)
        A = torch.empty(Hq).uniform_(0.5, 2.0, generator=g)
        if ties == 2:
            A[0] = 0.0
        W = torch.randn(Hq, Hkv * d if mode == 3 else d, generator=g) / (Hkv * d if mode == 3 else d) ** 0.5
        if ties == 1:
            W = (W * 8).round() / 8
        p = dma.problem(B, Hq, Hkv, L, d, w, flags=dma.DMA_FLAG_FULL_DELTA if mode == 3 else 0, causal=0 if mode == 2 else 1, dtype=dt)
        Vf = V.float().numpy()
        _, dl = oracle.delta_full(Vf, W.numpy(), A.numpy()) if mode == 3 else oracle.delta(Vf, W.numpy(), A.numpy(), Hq)
        weff, cu = min(w, L), None
        if mode == 1:
            cuts = sorted(set(int(c) for c in r.integers(1, max(2, L), int(r.integers(1, 12)) - 1) if 0 < c < L)) if L > 1 else []
            cu = [0] + cuts + [L]
            e = oracle.select_expiry_varlen(dl, weff, cu)
            got = dma.dma_mask_build_varlen(p, V.to(DEV), W.to(DEV), A.to(DEV), torch.tensor(cu, dtype=torch.int32, device=DEV))
        else:
            e = oracle.select_noncausal(dl, weff) if mode == 2 else oracle.select_expiry(dl, weff)
            got = dma.dma_mask_build(p, V.to(DEV), W.to(DEV), A.to(DEV))
        torch.cuda.synchronize()
        bias, expiry, bitmap = (t.cpu().numpy() for t in got)
        okd = np.array_equal(bias.view(np.uint32), dl.view(np.uint32))
        oke = np.array_equal(expiry, e)
        okb = mode == 2 or np.array_equal(bitmap.view(np.uint32), oracle.bitmap_from_expiry(e).view(np.uint32))
        if not (okd and oke and okb):
            T.fail(dict(B=B, Hq=Hq, Hkv=Hkv, L=L, w=w, d=d, mode=mode, ties=ties, dt=str(dt), cu=cu), "delta", okd, "expiry", oke, "bitmap", okb)
        T.n += 1


def decode(T):
    import test_gpu_decode as TDEC
    import test_gpu_decode_step as TSTEP
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 3, 4])), int(r.choice([1, 2, 4, 8]))
        d, B = int(r.choice([64, 128])), int(r.choice([1, 2, 3]))
        dtype = str(r.choice(["bf16", "fp32"]))
        try:
            if T.seed % 2:
                w = int(r.choice([1, 2, 5, 64, 127, 128, 129, 130, 257, 512, 1000]))
                n0 = int(r.choice([0, 1, w // 2, max(w - 1, 0), w, w + 1, w + 17, 3 * w, 5 * w + 3]))
                steps = int(r.integers(5, 30))
                case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=n0 + steps + int(r.integers(0, 9)), d=d, w=w, dtype=dtype, backward=False,
                                seed=T.seed, name="campaign decode-step")
                TSTEP.run(case, n0, steps, seed=T.seed, tie_head=bool(T.seed % 3 == 0))
            else:
                L = int(r.choice([1, 2, 31, 100, 255, 256, 257, 1000, 3001, 8192, 8193, 20000]))
                w = int(r.choice([1, 2, 7, 64, 100, 512, 2048, 30000]))
                case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, d=d, w=w, dtype=dtype, backward=False, seed=T.seed, name="campaign decode")
                TDEC.run_case(case, cap_extra=int(r.choice([0, 1, 8, 77])), seed=T.seed, tie_heads=bool(r.random() < 0.3))
        except AssertionError as ex:
            T.fail(case, repr(ex)[:300])
        T.n += 1


def chunk(T):
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 4])), int(r.choice([1, 2, 4]))
        L = int(r.choice([130, 257, 500, 1024, 1500, 2048, 3333, 5000]))
        w = int(r.choice([1, 31, 64, 129, 500, 1024, 6000]))
        d, B = int(r.choice([64, 128])), int(r.choice([1, 2]))
        dt = torch.bfloat16 if r.random() < 0.8 else torch.float32
        case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, dtype="bf16" if dt == torch.bfloat16 else "fp32", backward=False,
                        seed=T.seed, name="campaign chunk")
        inp = wl.make_inputs(case)
        Q, K, V = (inp[k].to(DEV) for k in ("Q", "K", "V"))
        p = dma.problem(B, case.Hq, Hkv, L, d, w, dtype=dt)
        bias, expiry, bitmap = dma.dma_mask_build(p, V, inp["W_delta"].to(DEV), inp["A"].to(DEV))
        O_full, lse_full = dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap)
        for _ in range(4):
            q_begin = int(r.integers(0, L))
            q_len = int(r.integers(1, L - q_begin + 1))
            O, lse = dma.dma_attn_fwd_chunk(p, q_begin, Q[:, q_begin:q_begin + q_len].contiguous(), K, V, bias, expiry)
            torch.cuda.synchronize()
            if not (close(O, O_full[:, q_begin:q_begin + q_len], 2e-2 if dt == torch.bfloat16 else 1e-4) and
                    close(lse, lse_full[:, :, q_begin:q_begin + q_len], 1e-3)):
                T.fail(dict(B=B, Hq=case.Hq, Hkv=Hkv, L=L, w=w, d=d, dt=str(dt), q_begin=q_begin, q_len=q_len))
            T.n += 1


def maskbwd(T):
    import test_gpu_delta_full as TDF
    import test_gpu_mask_bwd as TMB
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 3, 4])), int(r.choice([1, 2, 4, 8, 16]))
        d, B = int(r.choice([64, 128])), int(r.choice([1, 2, 3]))
        dtype = str(r.choice(["bf16", "fp32"]))
        L = int(r.choice([1, 3, 63, 64, 65, 127, 128, 129, 300, 517, 1024, 3000]))
        w = int(r.choice([1, 32, 128, 5000]))
        full = bool(T.seed % 2)
        if full and Hkv * G > 16:
            G = 2
        if Hkv * G > 32:
            G = 4
        case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, d=d, w=w, dtype=dtype, backward=True, seed=T.seed, name="campaign mask-bwd")
        try:
            (TDF.run_bwd if full else TMB.run_case)(case, seed=T.seed)
        except AssertionError as ex:
            T.fail(case, "full" if full else "per-head", repr(ex)[:300])
        T.n += 1


def strided_view(t, r):
    """a random strided placement of t [B, L, H, d] inside a larger buffer: (buffer, view holding t's values)"""
    B, L, H, d = t.shape
    l0, l1 = int(r.integers(0, 5)), int(r.integers(0, 9))
    hstep, h0, h1 = int(r.choice([1, 1, 2])), int(r.integers(0, 3)), int(r.integers(0, 2))
    big = torch.randn(B, l0 + L + l1, h0 + hstep * H + h1, d, device=DEV).to(t.dtype)
    v = big[:, l0:l0 + L, h0:h0 + hstep * H:hstep]
    v.copy_(t)
    return big, v


def strided(T):
    like = lambda buf, v: buf.as_strided(v.shape, v.stride(), v.storage_offset())
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 4])), int(r.choice([1, 2, 4]))
        L, w = int(r.choice([1, 130, 257, 512, 777, 1024, 2048])), int(r.choice([1, 31, 64, 129, 500, 3000]))
        d, B = int(r.choice([64, 128])), int(r.choice([1, 2]))
        dtn = str(r.choice(["bf16", "bf16", "bf16", "fp32"]))
        flags = int(r.choice([0, TILE, dma.DMA_FLAG_COMPACT_KV, dma.DMA_FLAG_SIMT])) if dtn == "bf16" else 0
        causal = int(r.random() < 0.8)
        case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, dtype=dtn, backward=True, seed=T.seed, name="campaign strided")
        inp = wl.make_inputs(case)
        Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
        W, A = inp["W_delta"].to(DEV), inp["A"].to(DEV) * (1.0 if causal else 0.25)
        mk = lambda: dma.problem(B, case.Hq, Hkv, L, d, w, dtype=case.torch_dtype, flags=flags if causal else flags & ~TILE, causal=causal)
        p0 = mk()
        m0 = dma.dma_mask_build(p0, V, W, A)
        O0, lse0 = dma.dma_attn_fwd(p0, Q, K, V, *m0)
        g0 = dma.dma_attn_bwd(p0, Q, K, V, O0, dO, lse0, *m0)
        (bq, Qv), (bk, Kv), (bv, Vv), (bo, dOv) = (strided_view(t, r) for t in (Q, K, V, dO))
        p = mk()
        for sdst, t in ((p.q_stride, Qv), (p.k_stride, Kv), (p.v_stride, Vv), (p.o_stride, dOv)):
            sdst[0], sdst[1], sdst[2] = t.stride(0), t.stride(1), t.stride(2)
        m1 = dma.dma_mask_build(p, Vv, W, A)
        Obuf, dQb, dKb, dVb = (torch.zeros_like(x) for x in (bo, bq, bk, bv))
        Ov, dQv, dKv, dVv = like(Obuf, dOv), like(dQb, Qv), like(dKb, Kv), like(dVb, Vv)
        O1, lse1 = dma.dma_attn_fwd(p, Qv, Kv, Vv, *m1, O=Ov)
        g1 = dma.dma_attn_bwd(p, Qv, Kv, Vv, O1, dOv, lse1, *m1, dQ=dQv, dK=dKv, dV=dVv)
        torch.cuda.synchronize()
        bad = [nm for nm, a, b in zip(("bias", "expiry", "bitmap", "O", "lse"), m0 + (O0, lse0), m1 + (O1, lse1)) if not torch.equal(a, b)]
        bad += [nm for nm, a, b in zip(("dQ", "dK", "dV", "dM"), g0, g1) if not close(b, a, 2e-2)]
        for nm, buf, v in (("O", Obuf, Ov), ("dQ", dQb, dQv), ("dK", dKb, dKv), ("dV", dVb, dVv)):
            tot, inside = float(buf.float().abs().sum()), float(v.float().abs().sum())
            if abs(tot - inside) > 1e-3 * max(1.0, tot):
                bad.append(nm + " written outside its view")
        if bad:
            T.fail(dict(B=B, Hq=case.Hq, Hkv=Hkv, L=L, w=w, d=d, dt=dtn, flags=flags, causal=causal), bad, [tuple(t.stride()) for t in (Qv, Kv, Vv, dOv)])
        T.n += 1


def host(T):
    import test_gpu_step_host as TH
    from helpers import gpu_run
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2, 4, 8])), int(r.choice([1, 2, 4]))
        L, w = int(r.choice([1, 100, 256, 333, 512, 1000, 2048])), int(r.choice([1, 17, 64, 300, 5000]))
        d, B, bwd = int(r.choice([64, 128])), int(r.choice([1, 2, 3])), bool(r.random() < 0.7)
        case = wl.small(C2, B=B, Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=d, dtype=str(r.choice(["bf16", "bf16", "fp32"])), backward=bwd, seed=T.seed,
                        name="campaign host step")
        inp = wl.make_inputs(case)
        try:
            got, dev = TH.host_step(case, inp), gpu_run(case, inp, backward=bwd)
            # where the library picks the token-compacted kernels (L >= 2048, 4 w <= L) and a KV head serves several query
            # heads, dK and dV are summed over the group with floating-point atomics: equal up to the order of the adds
            atomic = case.dtype == "bf16" and L >= 2048 and 4 * min(w, L) <= L and G > 1
            exact = ("O", "lse") + (("dK", "dV") if bwd and not atomic else ())
            bad = [k for k in exact if not torch.equal(got[k], dev[k].cpu())]
            if bwd:
                bad += [k for k in ("dQ", "dM") + (("dK", "dV") if atomic else ()) if not close(got[k], dev[k].cpu(), 2e-2)]
            if bad:
                T.fail(case, bad)
        except dma.DmaError as ex:
            T.fail(case, ex)
        T.n += 1


def large(T):
    from helpers import f64
    while T.running():
        r = T.next_rng()
        Hkv, G = int(r.choice([1, 2])), int(r.choice([1, 2, 4]))
        L = int(r.choice([8191, 12345, 16385, 20001, 30000, 40003, 65537]))
        w = int(r.choice([1, 100, 1024, 2048, 4097, 9000]))
        varlen = bool(r.random() < 0.4)
        if G * ((L + 127) // 128) * 2 > 8192:
            continue                                          # beyond the backward's step list (refused with DMA_ERR_UNSUPPORTED)
        case = wl.small(C2, B=1, Hq=Hkv * G, Hkv=Hkv, L=L, w=w, d=128, backward=True, seed=T.seed, name="campaign large")
        inp = wl.make_inputs(case)
        Q, K, V, dO = (inp[k].to(DEV) for k in ("Q", "K", "V", "dO"))
        W, A = inp["W_delta"].to(DEV), inp["A"].to(DEV)
        p_of = lambda flags: dma.problem(1, case.Hq, Hkv, L, 128, w, flags=flags)
        _, dl = oracle.delta(inp["V"].float().numpy(), inp["W_delta"].numpy(), inp["A"].numpy(), case.Hq)
        if varlen:
            cu = wl.packed_cu_seqlens(L, int(r.integers(2, 20)), seed=T.seed)
            mask = dma.dma_mask_build_varlen(p_of(0), V, W, A, torch.tensor(cu, dtype=torch.int32, device=DEV))
            e = oracle.select_expiry_varlen(dl, min(w, L), cu)
        else:
            mask = dma.dma_mask_build(p_of(0), V, W, A)
            e = oracle.select_expiry(dl, min(w, L))
        bad = []
        if not np.array_equal(mask[0].cpu().numpy().view(np.uint32), dl.view(np.uint32)):
            bad.append("delta")
        if not np.array_equal(mask[1].cpu().numpy(), e):
            bad.append("expiry")
        if not np.array_equal(mask[2].cpu().numpy().view(np.uint32), oracle.bitmap_from_expiry(e).view(np.uint32)):
            bad.append("bitmap")
        # the oracle first: sampled rows, and every row the sampled keys' gradients depend on (keys among the last 600, so only
        # the last 600 rows can keep them); its forward output on those rows, rounded to the element type, is the stored O
        # that both backward passes read
        edge = (L // 128) * 128
        tail = np.arange(max(0, L - 600), L)
        rows = np.unique(np.concatenate([r.integers(0, L, 6), [0, L - 1, edge - 1, min(L - 1, edge)], tail])).astype(np.int32)
        keys = np.unique(np.concatenate([r.integers(max(0, L - 600), L, 4), [L - 1]])).astype(np.int32)
        Q64, K64, V64, dO64 = (f64(inp[k]) for k in ("Q", "K", "V", "dO"))
        Or, lr = oracle.forward(Q64, K64, V64, dl.astype(np.float64), expiry=e, rows=rows)
        Ost = torch.from_numpy(Or).to(torch.bfloat16)
        Ofull = np.zeros_like(Q64)
        Ofull[:, rows] = f64(Ost)
        _, dKr, dVr, dMr = oracle.backward(Q64, K64, V64, dO64, dl.astype(np.float64), expiry=e, keys=keys, want_dq=False, O=Ofull)
        rows_t = torch.from_numpy(rows.astype(np.int64)).to(DEV)
        outs = []
        for flags in (TILE, dma.DMA_FLAG_COMPACT_KV):
            O, lse = dma.dma_attn_fwd(p_of(flags), Q, K, V, *mask)
            torch.cuda.synchronize()
            got = {"O": O.clone(), "lse": lse.clone()}
            O[:, rows_t] = Ost.to(DEV)
            lse[:, :, rows_t] = torch.from_numpy(lr.astype(np.float32)).to(DEV)
            g = dma.dma_attn_bwd(p_of(flags), Q, K, V, O, dO, lse, *mask)
            torch.cuda.synchronize()
            got.update(zip(("dQ", "dK", "dV", "dM"), g))
            outs.append(got)
        bad += ["tile against compacted: " + k for k in outs[0] if not close(outs[1][k], outs[0][k], 1e-3 if k == "lse" else 8e-2)]
        for o in outs:
            if np.abs(f64(o["O"][:, rows]) - Or).max() > 2e-2 * max(1.0, np.abs(Or).max()):
                bad.append("O rows")
            if np.abs(f64(o["lse"][:, :, rows]) - lr).max() > 1e-3 * max(1.0, np.abs(lr).max()):
                bad.append("lse rows")
            for nm, got, ref in (("dK", f64(o["dK"][:, keys]), dKr), ("dV", f64(o["dV"][:, keys]), dVr), ("dM", f64(o["dM"][:, :, keys]), dMr)):
                if np.abs(got - ref).max() > 2e-2 * max(1.0, np.abs(ref).max()):
                    bad.append(nm + " keys")
        if bad:
            T.fail(dict(Hq=case.Hq, Hkv=Hkv, L=L, w=w, varlen=varlen), bad)
        T.n += 1


CAMPAIGNS = {"attention": attention, "mask": mask, "decode": decode, "chunk": chunk, "maskbwd": maskbwd, "strided": strided,
             "host": host, "large": large}

if __name__ == "__main__":
    if len(sys.argv) < 2 or sys.argv[1] not in CAMPAIGNS:
        raise SystemExit(__doc__)
    if not torch.cuda.is_available():
        raise SystemExit("campaign.py needs a CUDA device")
    tally = Tally(sys.argv[1], float(sys.argv[2]) if len(sys.argv) > 2 else 300.0, int(sys.argv[3]) if len(sys.argv) > 3 else 5000)
    CAMPAIGNS[sys.argv[1]](tally)
    sys.exit(min(tally.done(), 255))
