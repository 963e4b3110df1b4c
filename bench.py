#!/usr/bin/env python
"""Benchmark of the DMA hot path (mask build + forward + backward) on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3] [--impl reference]

One step = dma_mask_build + dma_attn_fwd (+ dma_attn_bwd) on one batch of the workload (default: the 16K training
configuration the headline metric is quoted on). Prints one JSON line. With N > 1 (under torchrun) every rank
runs its own replica of the batch (the path has no exchange step), the step time is the max over ranks and the
value is the whole-job aggregate. `--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2508_02124_b200 import workloads as wl  # noqa: E402

METRIC = "dma_fwd_bwd_executed_tile_tflops"
NOMINAL_BF16_TFLOPS = 2250.0


def ncu_traffic(workload, kernel):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of a kernel on a workload, from the ncu captures
    summarised in profiles/dram_traffic.json; None where nothing was captured."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            return json.load(f).get(workload, {}).get(kernel)
    except (OSError, ValueError):
        return None


def algorithmic_bytes(case, kernel):
    """Lower bound of the HBM traffic of one launch: every input read once, every output written once."""
    e = 2 if case.dtype == "bf16" else 4
    q = case.B * case.L * case.Hq * case.d * e
    kv = case.B * case.L * case.Hkv * case.d * e
    rows = case.B * case.Hq * case.L * 4
    if kernel == "fwd":
        return 2 * q + 2 * kv + 3 * rows                      # Q, O; K, V; bias, expiry, lse
    return 2 * q + 2 * kv + 2 * kv + 4 * rows + 2 * case.B * case.L * case.Hq * case.d * 4   # Q, dO; K, V; dK, dV; bias, expiry, lse, D, dM; fp32 dQ accumulator read + written


def tile_flops(active_tiles, d, backward, bm=128, bn=128):
    """Executed-tile FLOPs: 2 GEMMs forward, 5 backward, each 2*bm*bn*d per active tile."""
    return active_tiles * (4 + (10 if backward else 0)) * bm * bn * d


def causal_tiles(case):
    T = -(-case.L // 128)
    return case.B * case.Hq * T * (T + 1) // 2


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        m = json.load(open(path))
        return {"bf16_burst": m["bf16_tflops"], "bf16_sustained": m.get("bf16_tflops_sustained", m["bf16_tflops"]),
                "hbm_gbs": m["hbm_gbs"], "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region (read-only query)."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                       "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.split(",") for r in open(self.f.name).read().strip().splitlines() if r.count(",") >= 6]
        os.unlink(self.f.name)
        if not rows:
            return out
        sm = sorted(float(r[0]) for r in rows)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        on = lambda r, k: "Active" in r[3 + k] and "Not" not in r[3 + k]
        reasons = [n for k, n in enumerate(names) if any(on(r, k) for r in rows)]
        out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=float(rows[0][1]), reasons=reasons, samples=len(rows),
                   power_w_max=max(float(r[2]) for r in rows), power_cap_frac=sum(on(r, 3) for r in rows) / len(rows))
        return out


def oracle_sample_run(case, inp, Ls):
    """The CPU oracle (fp32 instantiation, as it stands) on a bounded sample: the first KV-head group, first Ls
    rows (a causal prefix is a self-contained problem). Returns (seconds, executed-tile FLOPs of the sample)."""
    import oracle
    G = case.Hq // case.Hkv
    f = lambda t, n: np.ascontiguousarray(t[:1, :Ls, :n].float().numpy())
    Q, K, V, dO = f(inp["Q"], G), f(inp["K"], 1), f(inp["V"], 1), f(inp["dO"], G)
    W, A = inp["W_delta"][:G].numpy(), inp["A"][:G].numpy()
    t0 = time.perf_counter()
    _, dl = oracle.delta(V, W, A, G)
    e = oracle.select_expiry(dl, min(case.w, Ls))
    bmp = oracle.bitmap_from_expiry(e)
    oracle.forward(Q, K, V, dl, expiry=e, dtype=np.float32)
    if case.backward:
        oracle.backward(Q, K, V, dO, dl, expiry=e, dtype=np.float32)
    sec = time.perf_counter() - t0
    active = int(sum(bin(int(x)).count("1") for x in bmp.ravel()))
    return sec, tile_flops(active, case.d, case.backward), oracle.threads()


def run_reference(args, case):
    """--impl reference: the oracle on the host cores, each step one bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = wl.make_inputs(case)
    Ls = min(case.L, args.ref_rows)
    for _ in range(args.warmup):
        oracle_sample_run(case, inp, Ls)
    secs = []
    for _ in range(args.steps):
        s, flops, cores = oracle_sample_run(case, inp, Ls)
        secs.append(s)
    ms = 1e3 * sum(secs) / len(secs)
    val = flops / (ms * 1e-3) / 1e12
    sample = f"first KV-head group ({case.Hq // case.Hkv} query heads), first {Ls} rows of {case.name}, fp32 oracle, mask+fwd" + ("+bwd" if case.backward else "")
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                      "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": case.name, "sample": sample},
                      "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
                      "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="3", help="key of workloads.CONFIGS (3 = 16K training step, the headline)")
    ap.add_argument("--impl", default="dma", choices=["dma", "reference"])
    ap.add_argument("--ref-rows", type=int, default=4096, help="rows of the oracle sample per step (--impl reference)")
    ap.add_argument("--cpu-rows", type=int, default=16384, help="rows of the oracle sample for cpu_baseline (0 = skip)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--flags", type=int, default=0, help="dma_problem_t.flags (1 = ignore the bitmap, 2 = CUDA-core kernels)")
    ap.add_argument("--seq-len", type=int, default=0, help="override the workload's sequence length (profiling of a smaller case)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "dma" else args.warmup
    case = wl.CONFIGS[args.workload]
    if args.seq_len:
        case = wl.small(case, L=args.seq_len, w=min(case.w, args.seq_len), name=f"{case.name}-L{args.seq_len}")
    if args.impl == "reference":
        return run_reference(args, case)

    from paper_2508_02124_b200 import binding as dma
    from paper_2508_02124_b200 import replicas
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DMA path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    inp = wl.make_inputs(case)
    # the headline metric (TFLOP/s on executed tiles) is defined on the tile-walking kernels: DMA_FLAG_TILE_PATH; what the
    # library runs when left to choose is timed below as `best_path`
    tile_flag = dma.DMA_FLAG_TILE_PATH if not (args.flags & (dma.DMA_FLAG_COMPACT_KV | dma.DMA_FLAG_SIMT)) and case.causal else 0
    p = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, flags=args.flags | tile_flag)
    Q, K, V, dO, W, A = (inp[k].to(dev) for k in ("Q", "K", "V", "dO", "W_delta", "A"))
    m_ws, f_ws, b_ws = dma.dma_query_workspace(p)
    ws_m, ws_f, ws_b = (torch.empty(n, dtype=torch.uint8, device=dev) for n in (m_ws, f_ws, b_ws))
    bias = torch.empty(case.B, case.Hq, case.L, dtype=torch.float32, device=dev)
    expiry = torch.empty(case.B, case.Hq, case.L, dtype=torch.int32, device=dev)
    bitmap = torch.empty(dma.dma_bitmap_words(p), dtype=torch.int32, device=dev)
    O, lse = torch.empty_like(Q), torch.empty(case.B, case.Hq, case.L, dtype=torch.float32, device=dev)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    dM = torch.empty_like(lse)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    stage_ms = {"mask": 0.0, "fwd": 0.0, "bwd": 0.0}

    def step(timed=False):
        e = [ev() for _ in range(4)] if timed else None
        if timed: e[0].record()
        dma.dma_mask_build(p, V, W, A, bias, expiry, bitmap, ws_m)
        if timed: e[1].record()
        dma.dma_attn_fwd(p, Q, K, V, bias, expiry, bitmap, O, lse, ws_f)
        if timed: e[2].record()
        if case.backward:
            dma.dma_attn_bwd(p, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQ, dK, dV, dM, ws_b)
        if timed: e[3].record()
        return e

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    assert dma.dma_read_status(ws_f) == 0 and (not case.backward or dma.dma_read_status(ws_b) == 0), "device status"
    active = int(sum(bin(int(x) & 0xFFFFFFFF).count("1") for x in bitmap.cpu().numpy().ravel()))

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local]) if rank == 0 else None
    launches0 = dma.dma_launch_count()
    t0, t1 = ev(), ev()
    barrier()
    dma.dma_kernel_timing(True)            # event pairs around fwd_kernel / bwd_kernel alone (the library's measurement hook)
    t0.record()
    evs = [step(timed=True) for _ in range(args.steps)]
    t1.record()
    barrier()
    dma.dma_kernel_timing(False)
    kernel_ms = {"fwd": [], "bwd": []}
    for stage, t_ms in dma.dma_kernel_timing_read():
        kernel_ms[stage].append(t_ms)
    kernel_ms = {k: (sum(v) / len(v) if v else None) for k, v in kernel_ms.items()}
    launches = dma.dma_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = t0.elapsed_time(t1)
    for e in evs:
        stage_ms["mask"] += e[0].elapsed_time(e[1]); stage_ms["fwd"] += e[1].elapsed_time(e[2]); stage_ms["bwd"] += e[2].elapsed_time(e[3])
    stage_ms = {k: v / args.steps for k, v in stage_ms.items()}
    ms = replicas.max_over_ranks(total_ms / args.steps, dev)
    per_step = sorted(e[0].elapsed_time(e[3]) for e in evs)                 # each step's own span (events around its stages)
    step_stats = {"median_ms": per_step[len(per_step) // 2], "min_ms": per_step[0], "max_ms": per_step[-1]}
    # useful work: 4 d (forward) resp. 10 d (backward) flop per kept (row, key) pair, whatever the tile granularity
    kept_pairs = int((expiry.long() - torch.arange(case.L, device=dev)).clamp_(min=0).sum().item())
    useful_flops = kept_pairs * (4 + (10 if case.backward else 0)) * case.d

    # ---- mask-generation backward (bias gradient on to W_delta, A and V), timed on its own after the step: it is
    # not part of the headline metric. HBM-bound: V read once, dV read and written once, bias and dM read once.
    mask_bwd = None
    if case.backward:
        ws_g = torch.empty(dma.dma_mask_bwd_workspace(p), dtype=torch.uint8, device=dev)
        dWd, dAg = torch.empty_like(W), torch.empty_like(A)
        for _ in range(3):
            dma.dma_mask_bwd(p, V, W, A, bias, dM, dV, dWd, dAg, ws_g)
        g0, g1 = ev(), ev()
        barrier()
        g0.record()
        for _ in range(10):
            dma.dma_mask_bwd(p, V, W, A, bias, dM, dV, dWd, dAg, ws_g)
        g1.record()
        barrier()
        g_ms = g0.elapsed_time(g1) / 10
        g_bytes = 3 * V.numel() * V.element_size() + 2 * bias.numel() * 4
        mask_bwd = {"ms": g_ms, "algorithmic_bytes": g_bytes, "gbs": g_bytes / (g_ms * 1e-3) / 1e9}

    # ---- full sampling weights (DMA_FLAG_FULL_DELTA: W over all Hkv*d channels of the value row), timed on their own:
    # the mask build and its backward with a [Hq, Hkv*d] weight; 2 Hq Hkv d flop per key for z, three times that in the backward
    full_delta = None
    try:
        pf = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype,
                         flags=args.flags | dma.DMA_FLAG_FULL_DELTA)
        Wf = wl.full_delta_weights(case).to(dev)
        bias_f, exp_f, bmp_f = torch.empty_like(bias), torch.empty_like(expiry), torch.empty_like(bitmap)
        ws_fm = torch.empty(dma.dma_query_workspace(pf)[0], dtype=torch.uint8, device=dev)
        run_f = [lambda: dma.dma_mask_build(pf, V, Wf, A, bias_f, exp_f, bmp_f, ws_fm)]
        if case.backward:
            ws_fg = torch.empty(dma.dma_mask_bwd_workspace(pf), dtype=torch.uint8, device=dev)
            dWf, dAf = torch.empty_like(Wf), torch.empty_like(A)
            run_f.append(lambda: dma.dma_mask_bwd(pf, V, Wf, A, bias_f, dM, dV, dWf, dAf, ws_fg))
        times = []
        for f in run_f:
            for _ in range(3):
                f()
            g0, g1 = ev(), ev()
            barrier()
            g0.record()
            for _ in range(10):
                f()
            g1.record()
            barrier()
            times.append(g0.elapsed_time(g1) / 10)
        zflop = 2.0 * case.B * case.L * case.Hq * case.Hkv * case.d
        full_delta = {"mask_build_ms": times[0], "mask_bwd_ms": times[1] if len(times) > 1 else None, "z_gflop": zflop / 1e9}
    except dma.DmaError as e:
        full_delta = {"unsupported": str(e)}

    # ---- token-compacted forward (DMA_FLAG_COMPACT_KV), timed on its own: same outputs, O(L w d) work
    compact = None
    if case.dtype == "bf16" and case.d == 128 and not (args.flags & dma.DMA_FLAG_SIMT):
        pc = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype,
                         flags=args.flags | dma.DMA_FLAG_COMPACT_KV)
        ws_c = torch.empty(dma.dma_query_workspace(pc)[1], dtype=torch.uint8, device=dev)
        Oc, lsec = torch.empty_like(O), torch.empty_like(lse)
        for _ in range(3):
            dma.dma_attn_fwd(pc, Q, K, V, bias, expiry, bitmap, Oc, lsec, ws_c)
        c0, c1 = ev(), ev()
        barrier()
        c0.record()
        for _ in range(10):
            dma.dma_attn_fwd(pc, Q, K, V, bias, expiry, bitmap, Oc, lsec, ws_c)
        c1.record()
        barrier()
        assert dma.dma_read_status(ws_c) == 0, "device status (compact forward)"
        c_ms = c0.elapsed_time(c1) / 10
        compact = {"fwd_ms": c_ms, "tile_fwd_ms": stage_ms["fwd"], "fwd_speedup_over_tile_skipping": stage_ms["fwd"] / c_ms,
                   "max_abs_diff_vs_tile_path": float((Oc.float() - O.float()).abs().max())}
        if case.backward:
            ws_cb = torch.empty(dma.dma_query_workspace(pc)[2], dtype=torch.uint8, device=dev)
            dQc, dKc, dVc, dMc = torch.empty_like(dQ), torch.empty_like(dK), torch.empty_like(dV), torch.empty_like(dM)
            for _ in range(3):
                dma.dma_attn_bwd(pc, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQc, dKc, dVc, dMc, ws_cb)
            barrier()
            c0.record()
            for _ in range(10):
                dma.dma_attn_bwd(pc, Q, K, V, O, dO, lse, bias, expiry, bitmap, dQc, dKc, dVc, dMc, ws_cb)
            c1.record()
            barrier()
            assert dma.dma_read_status(ws_cb) == 0, "device status (compact backward)"
            cb_ms = c0.elapsed_time(c1) / 10
            compact.update({"bwd_ms": cb_ms, "tile_bwd_ms": stage_ms["bwd"], "bwd_speedup_over_tile_skipping": stage_ms["bwd"] / cb_ms,
                            "step_ms": stage_ms["mask"] + c_ms + cb_ms, "tile_step_ms": sum(stage_ms.values()),
                            "dK_max_abs_diff_vs_tile_path": float((dKc.float() - dK.float()).abs().max())})

    # ---- the step as a caller gets it with default flags: the library picks tile-walking or token-compacted kernels from the
    # descriptor (w against L); timed like the headline step, reported as wall time and as TFLOP/s on kept (row, key) pairs
    best_path = None
    if not (args.flags & (dma.DMA_FLAG_COMPACT_KV | dma.DMA_FLAG_TILE_PATH)):
        pa = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, flags=args.flags)
        sizes_a = dma.dma_query_workspace(pa)
        ws_am, ws_af, ws_ab = (torch.empty(n, dtype=torch.uint8, device=dev) for n in sizes_a)
        Oa, lsea = torch.empty_like(O), torch.empty_like(lse)
        dQa, dKa, dVa, dMa = torch.empty_like(dQ), torch.empty_like(dK), torch.empty_like(dV), torch.empty_like(dM)

        def step_a():
            dma.dma_mask_build(pa, V, W, A, bias, expiry, bitmap, ws_am)
            dma.dma_attn_fwd(pa, Q, K, V, bias, expiry, bitmap, Oa, lsea, ws_af)
            if case.backward:
                dma.dma_attn_bwd(pa, Q, K, V, Oa, dO, lsea, bias, expiry, bitmap, dQa, dKa, dVa, dMa, ws_ab)

        for _ in range(3):
            step_a()
        n_a = max(3, min(args.steps, 20))
        a0, a1 = ev(), ev()
        barrier()
        a0.record()
        for _ in range(n_a):
            step_a()
        a1.record()
        barrier()
        assert dma.dma_read_status(ws_af) == 0 and (not case.backward or dma.dma_read_status(ws_ab) == 0), "device status (default flags)"
        a_ms = replicas.max_over_ranks(a0.elapsed_time(a1) / n_a, dev)
        best_path = {"ms_per_step": a_ms, "path": "tile" if sizes_a[1] == dma.dma_query_workspace(p)[1] else "token-compacted",
                     "useful_tflops": world * useful_flops / (a_ms * 1e-3) / 1e12,
                     "speedup_over_tile_path": ms / a_ms, "max_abs_diff_O_vs_tile_path": float((Oa.float() - O.float()).abs().max())}

    # ---- the same tensors read as 12 documents packed along the sequence axis (dma_mask_build_varlen; the attention
    # kernels are unchanged): the bitmap becomes block-diagonal and tile skipping removes the other documents' tiles
    varlen = None
    if case.L >= 4096:
        cu = wl.packed_cu_seqlens(case.L, 12, seed=31)
        cu_t = torch.tensor(cu, dtype=torch.int32, device=dev)
        bias_v, exp_v, bmp_v = torch.empty_like(bias), torch.empty_like(expiry), torch.empty_like(bitmap)
        Ov, lsev = torch.empty_like(O), torch.empty_like(lse)
        stages = [lambda: dma.dma_mask_build_varlen(p, V, W, A, cu_t, bias_v, exp_v, bmp_v, ws_m),
                  lambda: dma.dma_attn_fwd(p, Q, K, V, bias_v, exp_v, bmp_v, Ov, lsev, ws_f)]
        if case.backward:
            stages.append(lambda: dma.dma_attn_bwd(p, Q, K, V, Ov, dO, lsev, bias_v, exp_v, bmp_v, dQ, dK, dV, dM, ws_b))
        v_ms = []
        for f in stages:
            for _ in range(3):
                f()
            g0, g1 = ev(), ev()
            barrier()
            g0.record()
            for _ in range(10):
                f()
            g1.record()
            barrier()
            v_ms.append(g0.elapsed_time(g1) / 10)
        # MMA-block skipping inside executed tiles (DMA_FLAG_BLOCK_SKIP): the same forward with the dead 16-key blocks of P V left out
        pbs = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, flags=p.flags | dma.DMA_FLAG_BLOCK_SKIP)
        bs_ms = None
        if case.dtype == "bf16" and case.d == 128 and not (args.flags & dma.DMA_FLAG_SIMT):
            for _ in range(3):
                dma.dma_attn_fwd(pbs, Q, K, V, bias_v, exp_v, bmp_v, Ov, lsev, ws_f)
            g0, g1 = ev(), ev()
            barrier()
            g0.record()
            for _ in range(10):
                dma.dma_attn_fwd(pbs, Q, K, V, bias_v, exp_v, bmp_v, Ov, lsev, ws_f)
            g1.record()
            barrier()
            bs_ms = g0.elapsed_time(g1) / 10
        act_v = int(sum(bin(int(x) & 0xFFFFFFFF).count("1") for x in bmp_v.cpu().numpy().ravel()))
        v_step = sum(v_ms)
        varlen = {"documents": 12, "lengths": [b - a for a, b in zip(cu, cu[1:])], "mask_ms": v_ms[0], "fwd_ms": v_ms[1],
                  "bwd_ms": v_ms[2] if case.backward else None, "step_ms": v_step, "active_tiles": act_v, "fwd_ms_block_skip": bs_ms,
                  "tflops_executed_tiles": tile_flops(act_v, case.d, case.backward) / (v_step * 1e-3) / 1e12}

    # ---- non-causal mode (causal = 0: every row of a head keeps the same min(w, L) keys; bf16 d = 128 runs token-compacted):
    # dense attention of L rows over w gathered keys per head
    noncausal = None
    if case.dtype == "bf16" and case.d == 128 and not (args.flags & dma.DMA_FLAG_SIMT):
        pn = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, causal=0, flags=args.flags)
        mn, fn_, bn_ = dma.dma_query_workspace(pn)
        ws_nm, ws_nf, ws_nb = (torch.empty(n, dtype=torch.uint8, device=dev) for n in (mn, fn_, bn_))
        bias_n, exp_n, bmp_n = torch.empty_like(bias), torch.empty_like(expiry), torch.empty_like(bitmap)
        On, lsen = torch.empty_like(O), torch.empty_like(lse)
        stages = [lambda: dma.dma_mask_build(pn, V, W, A, bias_n, exp_n, bmp_n, ws_nm),
                  lambda: dma.dma_attn_fwd(pn, Q, K, V, bias_n, exp_n, bmp_n, On, lsen, ws_nf)]
        if case.backward:
            stages.append(lambda: dma.dma_attn_bwd(pn, Q, K, V, On, dO, lsen, bias_n, exp_n, bmp_n, dQ, dK, dV, dM, ws_nb))
        n_ms = []
        for f in stages:
            for _ in range(3):
                f()
            g0, g1 = ev(), ev()
            barrier()
            g0.record()
            for _ in range(10):
                f()
            g1.record()
            barrier()
            n_ms.append(g0.elapsed_time(g1) / 10)
        assert dma.dma_read_status(ws_nf) == 0 and (not case.backward or dma.dma_read_status(ws_nb) == 0), "device status (non-causal)"
        keep = min(case.w, case.L)
        pair_flops = (4 + (10 if case.backward else 0)) * case.B * case.Hq * case.L * keep * case.d   # per kept (row, key) pair
        noncausal = {"mask_ms": n_ms[0], "fwd_ms": n_ms[1], "bwd_ms": n_ms[2] if case.backward else None, "step_ms": sum(n_ms),
                     "kept_keys_per_head": keep, "tflops_kept_pairs": pair_flops / (sum(n_ms) * 1e-3) / 1e12}

    # ---- prefill in pieces: the last 2048 rows of the sequence against all its keys (dma_attn_fwd_chunk), timed on its own
    chunk = None
    if case.dtype == "bf16" and case.d == 128 and case.L >= 4096 and not (args.flags & dma.DMA_FLAG_SIMT):
        q_len = 2048
        q_begin = case.L - q_len
        Qc = Q[:, q_begin:].contiguous()
        Oc2, lsec2 = torch.empty_like(Qc), torch.empty(case.B, case.Hq, q_len, dtype=torch.float32, device=dev)
        pcc = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype, flags=args.flags | dma.DMA_FLAG_COMPACT_KV)
        ws_ch = torch.empty(dma.dma_query_workspace(pcc)[1], dtype=torch.uint8, device=dev)
        for _ in range(3):
            dma.dma_attn_fwd_chunk(p, q_begin, Qc, K, V, bias, expiry, Oc2, lsec2, ws_ch)
        g0, g1 = ev(), ev()
        barrier()
        g0.record()
        for _ in range(10):
            dma.dma_attn_fwd_chunk(p, q_begin, Qc, K, V, bias, expiry, Oc2, lsec2, ws_ch)
        g1.record()
        barrier()
        ch_ms = g0.elapsed_time(g1) / 10
        chunk = {"q_begin": q_begin, "q_len": q_len, "ms": ch_ms,
                 "max_abs_diff_vs_full_forward": float((Oc2.float() - O[:, q_begin:].float()).abs().max())}

    # ---- one decoding step over this workload's K / V as the cache (dma_delta_range + dma_decode), timed on its own
    decode = None
    if rank == 0:
        pd = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype)
        dcache = torch.empty(case.B, case.Hq, case.L, dtype=torch.float32, device=dev)
        dma.dma_delta_range(pd, V, W, A, dcache, 0, case.L)
        qd = Q[:, -1].contiguous()
        od, lsed = torch.empty_like(qd), torch.empty(case.B, case.Hq, dtype=torch.float32, device=dev)
        ws_d = torch.empty(dma.dma_decode_workspace(pd), dtype=torch.uint8, device=dev)
        for _ in range(3):
            dma.dma_decode(pd, qd, K, V, dcache, od, lsed, None, False, ws_d)
        d0, d1 = ev(), ev()
        torch.cuda.synchronize()
        d0.record()
        for _ in range(20):
            dma.dma_decode(pd, qd, K, V, dcache, od, lsed, None, False, ws_d)
        d1.record()
        torch.cuda.synchronize()
        d_ms = d0.elapsed_time(d1) / 20
        keep = min(case.w, case.L)
        d_bytes = 2 * case.B * case.Hq * keep * case.d * K.element_size() + case.B * case.Hq * case.L * 4
        decode = {"us_per_step": d_ms * 1e3, "cached_keys": case.L, "kept_keys": keep, "algorithmic_bytes": d_bytes,
                  "gbs": d_bytes / (d_ms * 1e-3) / 1e9,
                  "dense_kv_read_bytes": 2 * case.B * case.Hkv * case.L * case.d * K.element_size()}
        # the same with the kept set carried from step to step (dma_decode_step): 24 consecutive steps that append the
        # workload's last 24 keys one at a time (delta of the new key + the step), the first 4 untimed
        n_inc = 24
        if case.L > n_inc + 1:
            probs = [dma.problem(case.B, case.Hq, case.Hkv, n, case.d, case.w, dtype=case.torch_dtype) for n in range(case.L - n_inc, case.L + 1)]
            for pp in probs:
                for sdst, ssrc in ((pp.k_stride, K.stride()), (pp.v_stride, V.stride())):
                    sdst[0], sdst[1], sdst[2] = ssrc[0], ssrc[1], ssrc[2]
            state = dma.dma_decode_state(probs[0], dev)
            dma.dma_decode_state_init(probs[0], dcache, state, ws_d)
            i0, i1 = ev(), ev()
            for t, pp in enumerate(probs[1:]):
                if t == 4:
                    torch.cuda.synchronize()
                    i0.record()
                dma.dma_delta_range(pp, V, W, A, dcache, pp.L - 1, pp.L)
                dma.dma_decode_step(pp, qd, K, V, dcache, state, od, lsed, ws_d)
            i1.record()
            torch.cuda.synchronize()
            inc_ms = i0.elapsed_time(i1) / (n_inc - 4)
            inc_bytes = 2 * case.B * case.Hq * keep * (case.d * K.element_size() + 4 + 4)      # K, V rows, delta and index of the kept keys
            decode.update({"incremental_us_per_step": inc_ms * 1e3, "incremental_algorithmic_bytes": inc_bytes,
                           "incremental_gbs": inc_bytes / (inc_ms * 1e-3) / 1e9})
            # the same two loops captured once in CUDA graphs and replayed: the device time without the host's launch cost
            # (seven and four small kernels per step: the eager numbers above are bound by the submission rate)
            try:
                g_full = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_full):
                    for _ in range(20):
                        dma.dma_decode(pd, qd, K, V, dcache, od, lsed, None, False, ws_d)
                dma.dma_decode_state_init(probs[0], dcache, state, ws_d)
                g_inc = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_inc):
                    for pp in probs[1:21]:
                        dma.dma_delta_range(pp, V, W, A, dcache, pp.L - 1, pp.L)
                        dma.dma_decode_step(pp, qd, K, V, dcache, state, od, lsed, ws_d)
                for name, gr, reinit in (("graph_us_per_step", g_full, False), ("incremental_graph_us_per_step", g_inc, True)):
                    ts = []
                    for _ in range(4):
                        if reinit:
                            dma.dma_decode_state_init(probs[0], dcache, state, ws_d)
                        torch.cuda.synchronize()
                        d0.record()
                        gr.replay()
                        d1.record()
                        torch.cuda.synchronize()
                        ts.append(d0.elapsed_time(d1) / 20)
                    decode[name] = min(ts[1:]) * 1e3
            except RuntimeError as e:          # capture refused: keep the eager numbers
                decode["graph_error"] = str(e)[:200]

    # ---- end to end through the host-buffer entry point: pinned host tensors in, results back on the host
    e2e = None
    if not args.no_e2e:
        arena = torch.empty(dma.dma_step_host_arena(p, case.backward), dtype=torch.uint8, device=dev)
        pin = lambda t: t.contiguous().pin_memory()
        hin = [pin(inp[k]) for k in ("Q", "K", "V", "dO", "W_delta", "A")]
        hO, hlse = pin(torch.empty_like(inp["Q"])), pin(torch.empty(case.B, case.Hq, case.L))
        hdQ, hdK, hdV, hdM = pin(torch.empty_like(inp["Q"])), pin(torch.empty_like(inp["K"])), pin(torch.empty_like(inp["V"])), pin(torch.empty(case.B, case.Hq, case.L))
        call = lambda: dma.dma_step_host(p, case.backward, hin[0], hin[1], hin[2], hin[3], hin[4], hin[5], hO, hlse, hdQ, hdK, hdV, hdM, arena)
        n_e2e = max(3, min(args.steps, 10))
        call(); call()
        barrier()
        t2, t3 = ev(), ev()
        t2.record()
        for _ in range(n_e2e):
            call()
        t3.record()
        barrier()
        e2e_ms = replicas.max_over_ranks(t2.elapsed_time(t3) / n_e2e, dev)
        nb = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts))
        h2d = nb(*hin) if case.backward else nb(hin[0], hin[1], hin[2], hin[4], hin[5])
        d2h = nb(hO, hlse) + (nb(hdQ, hdK, hdV, hdM) if case.backward else 0)
        assert torch.equal(hO, O.cpu()), "host-buffer path disagrees with the device path"
        e2e = {"value": world * tile_flops(active, case.d, case.backward) / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
               "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        # the same call with DMA_FLAG_COMPACT_KV (same outputs up to rounding, O(L w d) work): reported beside the headline
        if case.dtype == "bf16" and case.d == 128 and not (args.flags & dma.DMA_FLAG_SIMT):
            pce = dma.problem(case.B, case.Hq, case.Hkv, case.L, case.d, case.w, dtype=case.torch_dtype,
                              flags=args.flags | dma.DMA_FLAG_COMPACT_KV)
            arena_c = torch.empty(dma.dma_step_host_arena(pce, case.backward), dtype=torch.uint8, device=dev)
            call_c = lambda: dma.dma_step_host(pce, case.backward, hin[0], hin[1], hin[2], hin[3], hin[4], hin[5], hO, hlse, hdQ, hdK, hdV, hdM, arena_c)
            call_c(); call_c()
            barrier()
            t2.record()
            for _ in range(n_e2e):
                call_c()
            t3.record()
            barrier()
            e2e["compact_ms_per_step"] = replicas.max_over_ranks(t2.elapsed_time(t3) / n_e2e, dev)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    pk = peaks()
    flops = tile_flops(active, case.d, case.backward)
    value = world * flops / (ms * 1e-3) / 1e12
    dom = "bwd" if case.backward else "fwd"
    tensor_path = case.dtype == "bf16" and case.d == 128 and not (args.flags & dma.DMA_FLAG_SIMT)
    # Roofline of the dominant KERNEL (its own event pair, not the stage with its small pre / post kernels). The denominator
    # follows the clocks sampled during the timed region: the burst cuBLAS peak when the run was not power-capped (median SM
    # clock near the maximum, sw_power_cap active in a minority of samples), the sustained one otherwise; both fractions are printed.
    kflops = {"fwd": tile_flops(active, case.d, False), "bwd": tile_flops(active, case.d, False) * 2.5}
    capped = bool(clocks and clocks.get("sm_mhz") and (clocks["sm_mhz"] < 0.95 * clocks["sm_max_mhz"] or clocks.get("power_cap_frac", 0.0) > 0.5))
    peak_kind = "sustained" if capped else "burst"
    peak = pk["bf16_sustained"] if capped else pk["bf16_burst"]

    def kernel_roofline(kind):
        t_ms = kernel_ms.get(kind) or stage_ms[kind]
        ach = kflops[kind] / (t_ms * 1e-3) / 1e12
        return {"bound": "tensor" if tensor_path else "alu", "kernel": f"{kind}_kernel", "ms": t_ms,
                "timed": "event pair around the kernel alone" if kernel_ms.get(kind) else "stage time",
                "achieved": ach, "peak": peak, "peak_source": f"{pk['source']} {peak_kind} cuBLAS bf16 (chosen from the sampled clocks)",
                "unit": "TFLOP/s", "frac": ach / peak, "frac_burst": ach / pk["bf16_burst"], "frac_sustained": ach / pk["bf16_sustained"],
                "frac_nominal": ach / NOMINAL_BF16_TFLOPS,
                "traffic": ncu_traffic(case.name, kind + "_kernel") if tensor_path else None,
                "algorithmic_bytes": algorithmic_bytes(case, kind)}

    roofline = kernel_roofline(dom)
    if case.backward:
        roofline["forward"] = kernel_roofline("fwd")
    dom_flops = kflops[dom]
    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if case.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": case.name, "B": case.B, "Hq": case.Hq, "Hkv": case.Hkv, "L": case.L, "d": case.d, "w": case.w,
                   "passes": "mask+fwd+bwd" if case.backward else "mask+fwd", "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (no flush needed)" if (Q.numel() + 2 * K.numel()) * Q.element_size() > 126e6 else "inputs smaller than L2"},
        "stage_ms": stage_ms, "active_tiles": active, "causal_tiles": causal_tiles(case),
        "executed_tile_tflop_per_step": flops / 1e12,
        "frac_of_nominal_bf16_peak": value / world / NOMINAL_BF16_TFLOPS,
        "frac_of_measured_bf16_peak": value / world / peak, "measured_peak_used": peak_kind,
        "frac_of_measured_bf16_burst_peak": value / world / pk["bf16_burst"],
        "frac_of_measured_bf16_sustained_peak": value / world / pk["bf16_sustained"],
        "fwd_tflops": tile_flops(active, case.d, False) / (stage_ms["fwd"] * 1e-3) / 1e12,
        "bwd_tflops": (dom_flops / (stage_ms["bwd"] * 1e-3) / 1e12) if case.backward else None,
        "dense_causal_equivalent_speedup": causal_tiles(case) / max(active, 1),
        "roofline": roofline, "kernel_ms": kernel_ms,
        "gpu_launches": launches, "clocks": clocks, "e2e": e2e,
        "step_ms": step_stats, "kept_pairs": kept_pairs, "useful_tflop_per_step": useful_flops / 1e12,
        "useful_tflops": world * useful_flops / (ms * 1e-3) / 1e12,
    }
    if decode is not None:
        decode["frac_of_measured_hbm"] = decode["gbs"] / pk["hbm_gbs"]
        out["decode"] = decode
    if best_path is not None:
        out["best_path"] = best_path
    if compact is not None:
        out["compact"] = compact
    if full_delta is not None:
        out["full_delta"] = full_delta
    if varlen is not None:
        out["varlen"] = varlen
    if noncausal is not None:
        out["noncausal"] = noncausal
    if chunk is not None:
        out["fwd_chunk"] = chunk
    if mask_bwd is not None:
        mask_bwd["frac_of_measured_hbm"] = mask_bwd["gbs"] / pk["hbm_gbs"]
        out["mask_bwd"] = mask_bwd
    if args.cpu_rows:
        Ls = min(case.L, args.cpu_rows)
        sec, fl, cores = oracle_sample_run(case, inp, Ls)
        out["cpu_baseline"] = {"value": fl / sec / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "seconds": sec,
                               "sample": f"first KV-head group ({case.Hq // case.Hkv} query heads), first {Ls} rows of {case.name}, fp32 oracle"}
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
