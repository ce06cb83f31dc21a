"""Benchmark legs for the pieces around the headline path (used by bench.py --workload ...):

  a1_8b     one mini-batch of Algorithm 1 at 8B-class shapes (32 blocks, d = 4096, 32 heads of 128, 4096 tokens):
            64 conqur_step into the shared R_1 problem, 32 conqur_step_batched_range into the 1024 per-head problems,
            one batched update of those and one update of R_1
  hadamard  conqur_hadamard_rows on 32768 x 4096 bf16 (HBM-bound)
  fold      conqur_fold_weight, tensor-core mode: the MLP down projection of an 8B-class block, R_1^T W with
            W 4096 x 14336 (tensor-bound; three bf16 passes)

Each prints one JSON line in the layout of bench.py's headline line.
"""
from __future__ import annotations

import json
import os
import time

import numpy as np

from paper_2605_10793_b200 import dist as D
from paper_2605_10793_b200 import inputs as I


def _gen_site(args):
    name, kind, idx = args
    a = I.SITE_MODELS[name]
    if kind == "resid":
        return I.to_bf16_bits(I.batch(a.resid, idx))
    return I.to_bf16_bits(np.concatenate([I.batch(a.head, idx, problem=h) for h in range(a.n_heads)], axis=1))


def _pool_map(fn, jobs, world):
    workers = max(1, min(16, (os.cpu_count() or 2) // max(1, world)))
    if workers <= 1:
        return [fn(j) for j in jobs]
    import multiprocessing as mp
    with mp.get_context("fork").Pool(workers) as pool:
        return pool.map(fn, jobs, chunksize=1)


def run_algorithm1(args, g, ClockSampler, peaks):
    import torch
    from paper_2605_10793_b200 import algorithm1 as A1
    a = I.SITE_MODELS["a1_8b"]
    K, W = args.steps, max(args.warmup, 3)
    L, n = a.n_layers, a.n
    n_resid, n_o = 8, 4                                   # distinct activation matrices kept resident (32 MB each)
    t_gen = time.perf_counter()
    bits = _pool_map(_gen_site, [(a.name, "resid", i + 1000 * g.rank) for i in range(n_resid)] +
                     [(a.name, "o", i + 1000 * g.rank) for i in range(n_o)], g.world)
    t_gen = time.perf_counter() - t_gen
    host = [torch.from_numpy(b.view(np.int16)).pin_memory() for b in bits]
    dev = [h.cuda().view(torch.bfloat16) for h in host]
    resid, xo = dev[:n_resid], dev[n_resid:]
    cal = A1.Calibrator(a.d, a.n_heads, a.d_head, L, n, in_dtype="bf16", mode="tc")
    r1, r2 = I.site_initial_rotations(a)
    r1, r2 = torch.from_numpy(r1).cuda(), torch.from_numpy(r2).cuda()
    cal.set_rotations(r1, r2)

    def minibatch(src_resid, src_o):
        for l in range(L):
            cal.collect(l, src_resid[(2 * l) % n_resid], src_resid[(2 * l + 1) % n_resid], src_o[l % n_o])
        cal.end_minibatch()

    for _ in range(W):
        minibatch(resid, xo)
    if cal.ctx1.get_stats().status != 0 or cal.ctx2.get_stats().status != 0:
        raise SystemExit("warm-up failed")
    cal.set_rotations(r1, r2)
    cal.ctx1.set_profiling(False)
    cal.ctx2.set_profiling(False)
    sampler = ClockSampler(g.local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier(g)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(K):
        minibatch(resid, xo)
    e1.record()
    torch.cuda.synchronize()
    D.barrier(g)
    clocks = sampler.stop()
    ms = D.max_over_ranks(g, e0.elapsed_time(e1) / K)
    launches = cal.ctx1.get_profile()["total_launches"] + cal.ctx2.get_profile()["total_launches"]
    tokens = 3 * L * n                                    # activation rows entering a calibration site per mini-batch
    # breakdown of one mini-batch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    parts = []
    for _ in range(min(K, 3)):
        ev[0].record()
        for l in range(L):
            cal.collect(l, resid[(2 * l) % n_resid], resid[(2 * l + 1) % n_resid], xo[l % n_o])
        ev[1].record()
        cal.ctx2.update()
        ev[2].record()
        cal.ctx1.update()
        ev[3].record()
        torch.cuda.synchronize()
        parts.append([ev[i].elapsed_time(ev[i + 1]) for i in range(3)])
    parts = np.mean(np.array(parts), axis=0)
    # time of the head steps alone (same launches, nothing else in the stream)
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for l in range(L):
        cal.ctx2.step_batched_range(xo[l % n_o], n, a.n_heads * a.d_head, a.d_head, l * a.n_heads, a.n_heads)
    h1.record()
    torch.cuda.synchronize()
    head_steps_ms = h0.elapsed_time(h1)
    cal.ctx2.update()
    # end to end: every activation matrix comes from pinned host memory inside the timed region
    stage_r = [torch.empty_like(resid[0]) for _ in range(2)]
    stage_o = torch.empty_like(xo[0])
    cal.set_rotations(r1, r2)
    Ke = max(1, min(K, 4))
    torch.cuda.synchronize()
    e0.record()
    for _ in range(Ke):
        for l in range(L):
            stage_r[0].view(torch.int16).copy_(host[(2 * l) % n_resid], non_blocking=True)
            stage_r[1].view(torch.int16).copy_(host[(2 * l + 1) % n_resid], non_blocking=True)
            stage_o.view(torch.int16).copy_(host[n_resid + l % n_o], non_blocking=True)
            cal.collect(l, stage_r[0], stage_r[1], stage_o)
        jj, nn = cal.ctx1.get_objective()
        cal.end_minibatch()
    e1.record()
    torch.cuda.synchronize()
    ms_e2e = D.max_over_ranks(g, e0.elapsed_time(e1) / Ke)
    # roofline of the dominant kernel class of the mini-batch (the R_1 contractions at n = 4096)
    cal.ctx1.set_profiling(True)
    minibatch(resid, xo)
    torch.cuda.synchronize()
    prof = cal.ctx1.get_profile()
    cal.ctx1.set_profiling(False)
    classes = ["rotate_target", "accumulate", "ns_residual", "ns_poly", "ns_next"]
    dom = max(classes, key=lambda k: prof[k]["ms"])
    dn = max(1, prof[dom]["timed"])
    ach = prof[dom]["flops"] / (prof[dom]["ms"] * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]                      # launches timed alone between their own events: the burst figure
    st1, st2 = cal.ctx1.get_stats(), cal.ctx2.get_stats()
    if not g.is_main:
        D.finish(g)
        return 0
    out = {
        "metric": "calibration site-tokens/sec, one Algorithm-1 mini-batch at 8B-class shapes", "value": g.world * tokens / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": g.world, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{a.name}: {L} blocks, d={a.d}, {a.n_heads} heads x {a.d_head}, {n} tokens per mini-batch; per block 2 "
                               f"residual-stream sites into R_1 and one head-interleaved o_proj input into {a.n_heads} per-head problems",
                   "tokens_per_step": tokens, "mode": "tc",
                   "l2": f"{len(dev) * 32} MB of distinct activation matrices resident, cycled ({n_resid} residual, {n_o} o_proj)",
                   "input_gen_s": round(t_gen, 1)},
        "clocks": clocks,
        "e2e": {"value": g.world * tokens / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 3 * L * n * a.d * 2,
                "d2h_bytes_per_step": 16, "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
                     "kernel": f"tc_gemm_kernel, {dom} epilogue over the {2 * L} queued site matrices of {n} rows", "launches": dn,
                     "avg_launch_ms": prof[dom]["ms"] / dn, "peak_source": f"{peaks['source']} burst bf16",
                     "frac_of_sustained": ach / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": ach / 2250.0},
        "cpu_baseline": None,
        "breakdown_ms": {"site_steps": float(parts[0]), "heads_update": float(parts[1]), "r1_update": float(parts[2]),
                         "head_steps_alone": float(head_steps_ms)},
        "ns_steps_used": {"r1": int(st1.ns_steps_used), "heads": int(st2.ns_steps_used)},
    }
    print(json.dumps(out))
    D.finish(g)
    return 0


def run_hadamard(args, g, ClockSampler, peaks):
    import torch
    from paper_2605_10793_b200 import binding as B
    K, W = args.steps, max(args.warmup, 3)
    n, d = 32768, 4096
    x = torch.randn(n, d, device="cuda").to(torch.bfloat16)
    y = torch.empty_like(x)
    host = torch.empty((n, d), dtype=torch.bfloat16).pin_memory()
    host.copy_(x)
    for _ in range(W):
        B.conqur_hadamard_rows(x, out=y)
    sampler = ClockSampler(g.local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier(g)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(K):
        B.conqur_hadamard_rows(x, out=y)
    e1.record()
    torch.cuda.synchronize()
    D.barrier(g)
    clocks = sampler.stop()
    ms = D.max_over_ranks(g, e0.elapsed_time(e1) / K)
    Ke = max(1, min(K, 8))
    hout = torch.empty((n, d), dtype=torch.bfloat16).pin_memory()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(Ke):
        x.copy_(host, non_blocking=True)
        B.conqur_hadamard_rows(x, out=y)
        hout.copy_(y, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    ms_e2e = D.max_over_ranks(g, e0.elapsed_time(e1) / Ke)
    nbytes = 4.0 * n * d
    ach = nbytes / (ms * 1e-3) / 1e9
    from bench import ncu_traffic
    had_traffic, had_src = ncu_traffic("hadamard.hadamard_tc")
    if g.is_main:
        print(json.dumps({
            "metric": "rows/sec of the online Walsh-Hadamard transform at d=4096", "value": g.world * n / (ms * 1e-3), "unit": "rows/s",
            "n_gpus": g.world, "steps": K, "warmup": W, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"hadamard: {n} x {d} bf16 in, bf16 out", "l2": "256 MB in + 256 MB out per launch, larger than L2"},
            "clocks": clocks,
            "e2e": {"value": g.world * n / (ms_e2e * 1e-3), "unit": "rows/s", "h2d_bytes_per_step": int(nbytes / 2),
                    "d2h_bytes_per_step": int(nbytes / 2), "ms_per_step": ms_e2e},
            "gpu_launches": K,
            "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                         "traffic": (had_traffic * n / 16384) if had_traffic else None, "kernel": "hadamard_tc_kernel<bf16>",
                         "avg_launch_ms": ms,
                         "traffic_note": (f"dram read+write of an ncu capture at 16384 rows ({had_src}: the input read once, part of "
                                          "the output still in L2 at the end of the launch), scaled by the rows processed")
                                         if had_src else "no capture",
                         "bytes_per_launch": nbytes, "peak_source": peaks["source"]},
            "cpu_baseline": None}))
    D.finish(g)
    return 0


def run_fold(args, g, ClockSampler, peaks):
    import torch
    from paper_2605_10793_b200 import binding as B
    K, W = args.steps, max(args.warmup, 3)
    d, cols = 4096, 14336
    w = torch.from_numpy(I.random_weight(1, d, cols)).cuda()
    q, _ = np.linalg.qr(np.random.default_rng(2).standard_normal((d, d)))
    r = torch.from_numpy(q.astype(np.float32)).cuda()
    host = w.cpu().pin_memory()
    for _ in range(W):
        out = B.conqur_fold_weight(w, r, "output", "tc")
    sampler = ClockSampler(g.local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier(g)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(K):
        out = B.conqur_fold_weight(w, r, "output", "tc")
    e1.record()
    torch.cuda.synchronize()
    D.barrier(g)
    clocks = sampler.stop()
    ms = D.max_over_ranks(g, e0.elapsed_time(e1) / K)
    Ke = max(1, min(K, 4))
    hout = torch.empty_like(host)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(Ke):
        w.copy_(host, non_blocking=True)
        out = B.conqur_fold_weight(w, r, "output", "tc")
        hout.copy_(out, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    ms_e2e = D.max_over_ranks(g, e0.elapsed_time(e1) / Ke)
    flops = 3 * 2.0 * d * d * cols
    ach = flops / (ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]                      # launches timed alone between their own events: the burst figure
    if g.is_main:
        print(json.dumps({
            "metric": "weight elements folded/sec, R^T W with W 4096 x 14336 (whole call: split, three-pass product, status read)",
            "value": g.world * d * cols / (ms * 1e-3), "unit": "elements/s", "n_gpus": g.world, "steps": K, "warmup": W,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"fold: R_1^T W, W {d} x {cols} fp32 (an 8B-class MLP down projection), tensor-core mode",
                       "l2": "235 MB weight in, 235 MB out, larger than L2"},
            "clocks": clocks,
            "e2e": {"value": g.world * d * cols / (ms_e2e * 1e-3), "unit": "elements/s", "h2d_bytes_per_step": 4 * d * cols,
                    "d2h_bytes_per_step": 4 * d * cols, "ms_per_step": ms_e2e},
            "gpu_launches": 3 * K,
            "roofline": {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
                         "kernel": "tc_gemm_kernel, plain epilogue, 3 passes (timed with the two split kernels and the "
                                   "allocation of the output and scratch tensors of the call)",
                         "avg_launch_ms": ms, "flops_per_launch": flops, "peak_source": f"{peaks['source']} burst bf16",
                         "frac_of_sustained": ach / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": ach / 2250.0},
            "cpu_baseline": None}))
    D.finish(g)
    return 0


RUNNERS = {"a1_8b": run_algorithm1, "hadamard": run_hadamard, "fold": run_fold}
