#!/usr/bin/env python
"""Benchmark of the ConQuR calibration hot path on B200.

One "step" = one update cycle of the headline workload (d = 4096, batches of 2048 bf16 tokens, polar
update every 8 batches): 8 x conqur_step + 1 x conqur_update = 16384 tokens through every stage of the
path (row norms, rotate + corner target, cross-covariance accumulate, Newton-Schulz polar update with
its orthogonality check).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --workload c1|c3|c4a|c4a_zp|c4b|a1_8b|fold|hadamard      other workloads, same line layout
  python bench.py --profile-case path|heads|heads-timeline|hadamard [--d ..] [--n ..]    small bounded runs for profiler
                                                                            captures / the per-head kernel's timeline

N > 1 (torchrun): N independent replicas, one per GPU, no data-path collective ("weak" scaling).
--impl reference: times the float64 CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_10793_b200 import dist as D          # noqa: E402
from paper_2605_10793_b200 import inputs as I        # noqa: E402

METRIC = "calibration tokens/sec at d=4096 (whole path incl. polar update every 8 batches)"
WORKLOAD = "c2"
NOMINAL_BF16_TFLOPS = 2250.0          # B200 dense bf16 datasheet figure (context next to the measured peaks)


def ncu_traffic(tag: str):
    """DRAM bytes per launch of a kernel, as counted by a profiler capture: every summary under profiles/ carries
    lines `traffic <tag> <bytes>`; None when there is no capture of that kernel."""
    import glob
    import re
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        with open(path) as fh:
            for line in fh:
                m = re.match(r"\s*traffic\s+(\S+)\s+([0-9.eE+]+)\s*$", line)
                if m and m.group(1) == tag:
                    return float(m.group(2)), os.path.relpath(path, ROOT)
    return None, None


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            j = json.load(fh)
        return {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops"],
                "bf16_tflops_sustained": j.get("bf16_tflops_sustained", j["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def _gen_one(args):
    name, b, problem = args
    w = I.WORKLOADS[name]
    return I.to_bf16_bits(I.batch(w, b, problem=problem))


def generate_batches(name: str, count: int, replica: int, workers: int):
    """bf16 payloads (uint16, n x d) of the first `count` batches of the stream."""
    jobs = [(name, b, replica) for b in range(count)]
    if workers <= 1:
        return [_gen_one(j) for j in jobs]
    import multiprocessing as mp
    with mp.get_context("fork").Pool(workers) as pool:
        return pool.map(_gen_one, jobs, chunksize=1)


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 50 ms while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        # name the device by its UUID: under CUDA_VISIBLE_DEVICES the CUDA ordinal is not nvidia-smi's index
        self.gpu = str(gpu_index)
        try:
            import torch
            self.gpu = "GPU-" + str(torch.cuda.get_device_properties(gpu_index).uuid)
        except Exception:
            pass
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
def cpu_oracle_sample(w, cycles: int = 1, keep=None):
    """Time the float64 oracle, as it stands, on one update cycle of the workload (steps + one SVD update).
    keep: a dict that receives the first cycle's sign matrices, cross-covariance and objective (copied outside the
    timed sections) for the parity figures of the bench line."""
    from oracle import conqur_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count()])
    except Exception:
        threads = os.cpu_count()
    orc = O.OpuOracle(w.d, I.initial_rotation(w).astype(np.float64), quant_bits=w.quant_bits, prior_rel=w.prior_rel,
                      quant_mode=w.quant_mode, clip_ratio=w.clip_ratio)
    t_step = t_upd = 0.0
    for c in range(cycles):
        for b in range(w.update_every):
            x = I.batch(w, c * w.update_every + b).astype(np.float64)      # generation is not timed
            t0 = time.perf_counter()
            orc.step(x)
            t_step += time.perf_counter() - t0
            if keep is not None and c == 0:
                keep.setdefault("signs", []).append(orc.last_S.astype(np.int8))
        if keep is not None and c == 0:
            keep.update(M=orc.M.copy(), J=orc.J, N=orc.N)
        t0 = time.perf_counter()
        orc.update()
        t_upd += time.perf_counter() - t0
    cycle_s = (t_step + t_upd) / cycles
    return {"value": w.update_every * w.n / cycle_s, "unit": "tokens/s", "cores": int(threads), "kind": "oracle",
            "sample": f"{cycles} update cycle(s): {w.update_every} oracle steps of {w.n}x{w.d} "
                      f"({t_step / cycles:.2f} s) + 1 SVD update of {w.d}x{w.d} ({t_upd / cycles:.2f} s)",
            "step_s": t_step / (cycles * w.update_every), "update_s": t_upd / cycles}


def run_reference(args):
    g = D.Group(int(os.environ.get("RANK", "0")), 0, int(os.environ.get("WORLD_SIZE", "1")), False)
    if g.rank != 0:
        return 0
    w = I.WORKLOADS[WORKLOAD]
    # each reference "step" is a bounded sample of the cycle; keep the run within minutes
    steps = max(1, min(args.steps, 2))
    warm = 1 if args.warmup > 0 else 0
    if warm:
        cpu_oracle_sample(I.scaled(w, d=512, n=512), 1)
    samples = [cpu_oracle_sample(w, 1) for _ in range(steps)]
    best = max(samples, key=lambda s: s["value"])
    val = float(np.mean([s["value"] for s in samples]))
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * w.update_every * w.n / val, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": _workload_desc(w), "note": "float64 numpy oracle on host cores; bounded sample per step"},
        "cpu_baseline": {k: best[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    out["cpu_baseline"]["value"] = val
    print(json.dumps(out))
    return 0


def _gen_problem(args):
    name, p = args
    w = I.WORKLOADS[name]
    return I.to_bf16_bits(I.batch(w, 0, problem=p)), I.initial_rotation(w, p)


def run_batched(args, g, w):
    """The per-head workload (many independent d = 128 problems): one step = one batched conqur_step_batched over all
    problems + one batched conqur_update."""
    import torch
    from paper_2605_10793_b200 import binding as B
    K, W = args.steps, max(args.warmup, 3)
    P, n, d = w.problems, w.n, w.d
    workers = max(1, min(16, (os.cpu_count() or 2) // max(1, g.world)))
    t_gen = time.perf_counter()
    jobs = [(w.name, p + 100000 * g.rank) for p in range(P)]
    if workers > 1:
        import multiprocessing as mp
        with mp.get_context("fork").Pool(workers) as pool:
            gen = pool.map(_gen_problem, jobs, chunksize=8)
    else:
        gen = [_gen_problem(j) for j in jobs]
    t_gen = time.perf_counter() - t_gen
    host = torch.from_numpy(np.concatenate([b for b, _ in gen], axis=0).view(np.int16)).pin_memory()
    dev = host.cuda().view(torch.bfloat16)
    r0 = torch.from_numpy(np.stack([r for _, r in gen])).cuda()
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P, quant_bits=w.quant_bits, prior_rel=w.prior_rel,
                    quant_mode=w.quant_mode, clip_ratio=w.clip_ratio)

    def one(x):
        ctx.set_R(r0)            # every step is the workload's single (step, update) from R0; set_R is outside the metric's work
        ctx.step_batched(x, n, d, n * d)
        ctx.update()

    for _ in range(W):
        one(dev)
    if ctx.get_stats().status != 0:
        raise SystemExit("warm-up failed")
    sampler = ClockSampler(g.local_rank)
    sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    D.barrier(g)
    torch.cuda.synchronize()
    ctx.set_profiling(False)
    for k in range(K):
        ctx.set_R(r0)
        ev[k][0].record()
        ctx.step_batched(dev, n, d, n * d)
        ev[k][1].record()
        ctx.update()
        ev[k][2].record()
    torch.cuda.synchronize()
    D.barrier(g)
    clocks = sampler.stop()
    launches = ctx.get_profile()["total_launches"]
    step_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    upd_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    ms = D.max_over_ranks(g, step_ms + upd_ms)
    tokens = P * n
    value = g.world * tokens / (ms * 1e-3)
    # end to end: the batch comes from pinned host memory inside the timed region, the objectives go back
    stage = torch.empty_like(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for k in range(K):
        stage.view(torch.int16).copy_(host, non_blocking=True)
        ctx.set_R(r0)
        ctx.step_batched(stage, n, d, n * d)
        jj, nn = ctx.get_objective()
        ctx.update()
    e1.record()
    torch.cuda.synchronize()
    ms_e2e = D.max_over_ranks(g, e0.elapsed_time(e1) / K)
    st = ctx.get_stats()
    peaks = _peaks()
    step_bytes = 2.0 * P * n * d
    ach = step_bytes / (step_ms * 1e-3) / 1e9
    heads_traffic, heads_src = ncu_traffic("c4b.tcb_step")
    if not g.is_main:
        D.finish(g)
        return 0
    out = {
        "metric": "calibration tokens/sec, 1024 independent d=128 problems (one batched step + one batched polar update)",
        "value": value, "unit": "tokens/s", "n_gpus": g.world, "steps": K, "warmup": W, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: {P} problems x ({n} x {d}) bf16, Student-t(3), 2 outlier channels x100, R0 randomised "
                               "Hadamard per problem", "tokens_per_step": tokens, "mode": "tc, fused per-head kernels",
                   "l2": f"inputs larger than L2: {dev.numel() * 2 / 1e6:.0f} MB read once per step", "input_gen_s": round(t_gen, 1)},
        "clocks": clocks,
        "e2e": {"value": g.world * tokens / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": int(dev.numel() * 2),
                "d2h_bytes_per_step": 16 * P, "ms_per_step": ms_e2e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                     "traffic": (heads_traffic * (P * n) / (592 * 2048)) if heads_traffic else None, "kernel": "tcb_step_kernel",
                     "avg_launch_ms": step_ms,
                     "traffic_note": (f"dram read+write of an ncu capture at 592 problems x 2048 tokens ({heads_src}), scaled by the "
                                      "tokens processed: the kernel streams its input once") if heads_src else "no capture",
                     "bytes_per_launch": step_bytes, "peak_source": peaks["source"],
                     "tensor_tflops": 4.0 * P * n * d * d / (step_ms * 1e-3) / 1e12},
        "cpu_baseline": None,
        "step_ms": step_ms, "polar_update_ms": upd_ms, "ns_steps_used": int(st.ns_steps_used), "orth_err": float(st.orth_err),
    }
    print(json.dumps(out))
    D.finish(g)
    return 0


def _workload_desc(w):
    return (f"{w.name}: d={w.d}, {w.n_batches} batches x {w.n} tokens, bf16 Student-t(3) with {w.n_outlier} outlier "
            f"channels x{w.outlier_scale:g}, {w.n_massive_rows} massive tokens x{w.massive_scale:g}/batch, "
            f"R0=randomised Hadamard, polar update every {w.update_every} batches")


def parity_sample(ctx, w, r0, dev, keep):
    """The first cycle of the stream through the library once more, compared with what the oracle's timed sample of
    the same cycle left behind: fraction of sign decisions that differ, raw cross-covariance and objective error."""
    import torch
    cyc = w.update_every
    ctx.set_R(r0)
    for b in range(cyc):
        ctx.step(dev[b])
    j, n = ctx.get_objective()
    m = ctx.get_M().cpu().numpy().astype(np.float64)
    s_gpu = ctx.debug_get_signs(cyc * w.n).cpu().numpy()
    s_ref = np.concatenate(keep["signs"], axis=0)
    ctx.update()
    torch.cuda.synchronize()
    return {"what": f"cycle 1 ({cyc} batches from R0) against the float64 oracle",
            "sign_flip_fraction": float((s_gpu != s_ref).mean()),
            "M_rel_raw": float(np.linalg.norm(m - keep["M"]) / np.linalg.norm(keep["M"])),
            "J_rel": float(abs(j - keep["J"]) / keep["J"]), "N_equal": bool(n == keep["N"])}


def heads_entry(peaks, K: int = 10, W: int = 3):
    """The per-head workload (1024 problems of d = 128, 4096 tokens each) inside the headline run: one batched step and
    one batched update, device-timed.  64 distinct seeded problems, stored 16 times at distinct addresses (every byte
    is still read from HBM once per step)."""
    import torch
    from paper_2605_10793_b200 import binding as B
    w = I.WORKLOADS["c4b"]
    P, n, d, distinct = w.problems, w.n, w.d, 64
    gen = [_gen_problem((w.name, p)) for p in range(distinct)]
    x = torch.from_numpy(np.concatenate([b for b, _ in gen], axis=0).view(np.int16)).cuda().view(torch.bfloat16)
    x = x.repeat(P // distinct, 1).contiguous()
    r0 = torch.from_numpy(np.stack([r for _, r in gen])).cuda().repeat(P // distinct, 1, 1).contiguous()
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    for k in range(W + K):
        ctx.set_R(r0)
        e = ev[max(0, k - W)]
        e[0].record()
        ctx.step_batched(x, n, d, n * d)
        e[1].record()
        ctx.update()
        e[2].record()
    torch.cuda.synchronize()
    st = ctx.get_stats()
    step_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    upd_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    gbs = 2.0 * P * n * d / (step_ms * 1e-3) / 1e9
    ctx.close()
    return {"workload": f"c4b: {P} problems x ({n} x {d}) bf16", "step_ms": step_ms, "polar_update_ms": upd_ms,
            "tokens_per_s": P * n / ((step_ms + upd_ms) * 1e-3), "step_hbm_gbs": gbs, "step_frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
            "ns_steps_used": int(st.ns_steps_used), "status": int(st.status)}


def hadamard_entry(peaks, K: int = 20, W: int = 3):
    """conqur_hadamard_rows on 32768 x 4096 bf16 -> bf16 inside the headline run, device-timed."""
    import torch
    from paper_2605_10793_b200 import binding as B
    n, d = 32768, 4096
    x = torch.randn(n, d, device="cuda").to(torch.bfloat16)
    y = torch.empty_like(x)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for k in range(W + K):
        if k == W:
            e0.record()
        B.conqur_hadamard_rows(x, out=y)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / K
    gbs = 4.0 * n * d / (ms * 1e-3) / 1e9
    return {"workload": f"hadamard: {n} x {d} bf16 in, bf16 out", "ms": ms, "hbm_gbs": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
            "status": int(B.conqur_hadamard_status())}


def profile_case(args):
    """A small, bounded invocation for profiler captures: a few dozen launches, well under a few GB on the device.
    Prints what it ran so that a plain run can be checked before a capture.
      path      --batches B batches of --n tokens at width --d through conqur_step (queued, one run of the two
                products) and one conqur_update
      heads     the per-head kernels: --problems problems of d = 128, --n tokens each, two (step, update) rounds
      heads-timeline  the per-head step kernel's own timestamps (conqur_debug_trace_heads): thread block 0, tiles of
                its second problem, SM cycles relative to the first event shown
      hadamard  conqur_hadamard_rows on --n x --d bf16, three launches"""
    import torch
    from paper_2605_10793_b200 import binding as B
    if args.profile_case == "hadamard":
        x = torch.randn(args.n, args.d, device="cuda").to(torch.bfloat16)
        y = torch.empty_like(x)
        for _ in range(3):
            B.conqur_hadamard_rows(x, out=y, cuda_cores_only=args.cuda_cores_only)
        rc = B.conqur_hadamard_status()
        print(f"profile-case hadamard n={args.n} d={args.d} bf16: status={rc} |y|max={y.float().abs().max().item():.3f}")
        return 0 if rc == 0 else 1
    if args.profile_case == "heads-timeline":
        P, n, d = args.problems, args.n, 128
        x = (torch.randn(P * n, d, device="cuda") * (1.0 + 20.0 * (torch.arange(d, device="cuda") < 2))).to(torch.bfloat16)
        ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P)
        for _ in range(3):
            ctx.step_batched(x, n, d, n * d)
        trace = torch.zeros(96 * 16, dtype=torch.int64, device="cuda")
        ctx.debug_trace_heads(trace)
        ctx.step_batched(x, n, d, n * d)
        ctx.debug_trace_heads(None)
        t = trace.cpu().numpy().reshape(96, 16)
        tiles = (n + 127) // 128
        names = ["copy", "mma1", "mma2", "norm>", "norm<", "epi>", "norms", "cfree", "y", "ld0", "st0", "ld1", "epi<", "out?", "out>", "out<"]
        order = [0, 1, 2, 3, 4, 5, 6, 7, 8, 13, 14, 15, 9, 10, 11, 12]
        first = tiles if 2 * tiles <= 96 else 0                       # the second problem of the block: steady state
        t0 = t[first, 0]
        print(f"profile-case heads-timeline P={P} n={n}: block 0, tiles {first}..{min(96, first + tiles) - 1} "
              f"(problem boundary after tile {first + tiles - 1}), SM cycles since the first copy shown")
        print(" tile " + " ".join(f"{nm:>7s}" for nm in names))
        for i in range(first, min(96, first + tiles + 3)):
            print(f"{i:5d} " + " ".join(f"{(t[i, e] - t0) if t[i, e] else 0:7d}" for e in order))
        st = ctx.get_stats()
        return 0 if st.status == 0 else 1
    if args.profile_case == "heads":
        P, n, d = args.problems, args.n, 128
        x = (torch.randn(P * n, d, device="cuda") * (1.0 + 20.0 * (torch.arange(d, device="cuda") < 2))).to(torch.bfloat16)
        ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P)
        for _ in range(2):
            ctx.step_batched(x, n, d, n * d)
            ctx.update()
        st = ctx.get_stats()
        print(f"profile-case heads P={P} n={n}: ns_steps={st.ns_steps_used} orth={st.orth_err:.2e} status={st.status}")
        return 0 if st.status == 0 else 1
    d, n, nb = args.d, args.n, max(1, args.batches)
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, r0="hadamard" if d & (d - 1) == 0 else "qr")
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", defer_batches=nb,
                    prior_rel=0.0 if nb * n >= 2 * d else 1e-2, debug_flags=B.CONQUR_DEBUG_NO_GRAPH)
    ctx.set_R(torch.from_numpy(I.initial_rotation(w)).cuda())
    xs = [torch.from_numpy(I.batch(w, b)).cuda().to(torch.bfloat16) for b in range(nb)]
    torch.cuda.synchronize()
    for x in xs:
        ctx.step(x)
    j, cnt = ctx.get_objective()
    ctx.update()
    st = ctx.get_stats()
    print(f"profile-case path d={d} n={n} batches={nb}: J/N={j / cnt:.5f} ns_steps={st.ns_steps_used} "
          f"orth={st.orth_err:.2e} status={st.status} launches={ctx.get_profile()['total_launches']}")
    return 0 if st.status == 0 else 1


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--distinct-cycles", type=int, default=0, help="cycles of distinct batches kept resident (0=all)")
    ap.add_argument("--no-extra", action="store_true", help="skip the per-head and Walsh-Hadamard entries of the line")
    ap.add_argument("--profile-case", default=None, choices=["path", "heads", "heads-timeline", "hadamard"],
                    help="run a small bounded case (for profiler captures) instead of the benchmark")
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--n", type=int, default=2048)
    ap.add_argument("--problems", type=int, default=592)
    ap.add_argument("--batches", type=int, default=1, help="--profile-case path: batches queued before the products run")
    ap.add_argument("--no-graph", action="store_true", help="enqueue the update's launches directly (profiler launch lists)")
    ap.add_argument("--cuda-cores-only", action="store_true", help="--profile-case hadamard: the CUDA-core kernel")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.profile_case:
        return profile_case(args)

    import torch
    from paper_2605_10793_b200 import binding as B
    g = D.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(g.local_rank)
    B.load()
    if args.workload not in I.WORKLOADS:
        import bench_extra as X      # Algorithm-1 mini-batch, Hadamard transform, weight folding
        return X.RUNNERS[args.workload](args, g, ClockSampler, _peaks())
    w = I.WORKLOADS[args.workload]
    if w.problems > 1:
        return run_batched(args, g, w)
    K, W = args.steps, max(args.warmup, 3)
    cyc = w.update_every
    total_cycles = w.n_batches // cyc
    distinct = min(total_cycles, args.distinct_cycles or total_cycles, max(K, 1))
    n_batches = distinct * cyc
    workers = max(1, min(16, (os.cpu_count() or 2) // max(1, g.world)))
    t_gen = time.perf_counter()
    bits = generate_batches(w.name, n_batches, g.rank, workers)
    t_gen = time.perf_counter() - t_gen

    # inputs: pinned host copies (for the end-to-end leg) and resident device copies (for the device-timed leg)
    host = [torch.from_numpy(b.view(np.int16)).pin_memory() for b in bits]
    dev = [h.cuda(non_blocking=True).view(torch.bfloat16) for h in host]
    torch.cuda.synchronize()
    resident_bytes = sum(t.numel() * 2 for t in dev)
    r0 = torch.from_numpy(I.initial_rotation(w)).cuda()

    # the products of a cycle run once over all its batches (conqur_config.defer_batches = the update cadence)
    ctx = B.Context(d=w.d, n_max=w.n, in_dtype="bf16", mode="tc", quant_bits=w.quant_bits, prior_rel=w.prior_rel,
                    quant_mode=w.quant_mode, clip_ratio=w.clip_ratio, defer_batches=cyc, ns_steps=w.ns_steps,
                    debug_flags=B.CONQUR_DEBUG_NO_GRAPH if args.no_graph else 0)
    ctx.set_R(r0)

    def cycle_resident(c):
        base = (c % distinct) * cyc
        for b in range(cyc):
            ctx.step(dev[base + b])
        ctx.update()

    for c in range(W):
        cycle_resident(c)
    st = ctx.get_stats()
    if st.status != 0:
        raise SystemExit(f"warm-up failed: {B.strerror(st.status)}")
    ctx.set_R(r0)

    # ---------------- device-timed leg: inputs resident in HBM
    ctx.set_profiling(False)                     # resets the launch counters
    sampler = ClockSampler(g.local_rank)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    D.barrier(g)
    torch.cuda.synchronize()
    ev0.record()
    for c in range(K):
        cycle_resident(c)
    ev1.record()
    torch.cuda.synchronize()
    D.barrier(g)
    ms_local = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    launches = ctx.get_profile()["total_launches"]
    st = ctx.get_stats()
    j_last, n_last = st.last_J, st.last_N
    ms = D.max_over_ranks(g, ms_local)
    tokens = K * cyc * w.n
    value = g.world * tokens / (ms * 1e-3)

    # ---------------- end-to-end leg: host buffers, H2D inside the timed region, objective read back each cycle
    e2e = None
    if not args.no_e2e:
        ctx.set_R(r0)
        ring = 2 * cyc
        stage = [torch.empty((w.n, w.d), dtype=torch.bfloat16, device="cuda") for _ in range(ring)]
        copy_stream = torch.cuda.Stream()
        ready = [torch.cuda.Event() for _ in range(ring)]
        freed = [torch.cuda.Event() for _ in range(ring)]
        main_stream = torch.cuda.current_stream()

        def enqueue_copy(i):
            slot = i % ring
            with torch.cuda.stream(copy_stream):
                if i >= ring:
                    copy_stream.wait_event(freed[slot])
                stage[slot].view(torch.int16).copy_(host[i % n_batches], non_blocking=True)
                ready[slot].record(copy_stream)

        # the cycle's result (objective sum and token count) goes to page-locked host memory through the stream and is
        # looked at one cycle later, so the read never drains the queue
        res_j = [torch.zeros(1, dtype=torch.float64).pin_memory() for _ in range(2)]
        res_n = [torch.zeros(1, dtype=torch.int64).pin_memory() for _ in range(2)]
        res_ev = [torch.cuda.Event() for _ in range(2)]
        objective_log = []

        def collect(c):
            res_ev[c % 2].synchronize()
            objective_log.append((float(res_j[c % 2][0]), int(res_n[c % 2][0])))

        total_b = K * cyc
        D.barrier(g)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_wall = time.perf_counter()
        e0.record()
        issued = 0
        while issued < min(ring, total_b):
            enqueue_copy(issued); issued += 1
        for i in range(total_b):
            slot = i % ring
            main_stream.wait_event(ready[slot])
            ctx.step(stage[slot])
            freed[slot].record(main_stream)
            if issued < total_b:
                enqueue_copy(issued); issued += 1
            if (i + 1) % cyc == 0:
                c = (i + 1) // cyc - 1
                if c >= 2:
                    collect(c - 2)                     # frees this cycle's result slot
                ctx.get_objective_async(res_j[c % 2], res_n[c % 2])
                res_ev[c % 2].record(main_stream)
                ctx.update()
        for c in range(max(0, K - 2), K):
            collect(c)
        e1.record()
        torch.cuda.synchronize()
        assert len(objective_log) == K and all(0 < n_ <= cyc * w.n and j_ > 0 for j_, n_ in objective_log), objective_log[:4]
        t_wall = time.perf_counter() - t_wall
        D.barrier(g)
        ms_e2e = D.max_over_ranks(g, max(e0.elapsed_time(e1), 0.0))
        e2e = {"value": g.world * tokens / (ms_e2e * 1e-3), "unit": "tokens/s",
               "h2d_bytes_per_step": cyc * w.n * w.d * 2, "d2h_bytes_per_step": 16,
               "ms_per_step": ms_e2e / K, "host_wall_ms_per_step": 1e3 * t_wall / K,
               "how": "pinned host batches -> double-buffered cudaMemcpyAsync on a copy stream -> conqur_step; "
                      "objective and token count of every cycle read back through the stream (conqur_get_objective_async) "
                      "and checked on the host one cycle later"}
        del stage

    # ---------------- breakdown pass (no per-launch events): the 8 steps and the update of a cycle timed apart
    ctx.set_R(r0)
    step_ms, upd_ms = [], []
    for c in range(min(K, 4)):
        base = (c % distinct) * cyc
        u0, u1, u2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        u0.record()
        for b in range(cyc):
            ctx.step(dev[base + b])
        u1.record()
        ctx.update()
        u2.record()
        torch.cuda.synchronize()
        step_ms.append(u0.elapsed_time(u1))
        upd_ms.append(u1.elapsed_time(u2))

    # ---------------- roofline pass: same workload, each contraction launch bracketed by CUDA events
    ctx.set_R(r0)
    ctx.set_profiling(True)
    for c in range(min(K, 4)):
        base = (c % distinct) * cyc
        for b in range(cyc):
            ctx.step(dev[base + b])
        ctx.update()
        torch.cuda.synchronize()
    prof = ctx.get_profile()
    st2 = ctx.get_stats()
    ctx.set_profiling(False)
    peaks = _peaks()
    gemm_classes = ["rotate_target", "accumulate", "ns_residual", "ns_poly", "ns_next"]
    tot_fl = sum(prof[k]["flops"] for k in gemm_classes)
    tot_ms = sum(prof[k]["ms"] for k in gemm_classes)
    tot_n = sum(prof[k]["timed"] for k in gemm_classes)
    # every launch is timed alone between its own events and the SM clock stays near its maximum over the short
    # timed region, so the burst figure is the denominator (the sustained one is given beside it)
    peak = peaks["bf16_tflops"]
    detail = {k: {"launches": prof[k]["timed"], "avg_ms": prof[k]["ms"] / max(1, prof[k]["timed"]),
                  "tflops": (prof[k]["flops"] / (prof[k]["ms"] * 1e-3) / 1e12) if prof[k]["ms"] > 0 else 0.0}
              for k in gemm_classes}
    for k in gemm_classes:
        detail[k]["frac_of_measured_burst"] = detail[k]["tflops"] / peaks["bf16_tflops"]
        detail[k]["frac_of_nominal_2250"] = detail[k]["tflops"] / NOMINAL_BF16_TFLOPS
    # the dominant kernel: the instantiation of tc_gemm_kernel with the largest share of device time
    dom = max(gemm_classes, key=lambda k: prof[k]["ms"])
    dom_fl, dom_ms, dom_n = prof[dom]["flops"], prof[dom]["ms"], max(1, prof[dom]["timed"])
    achieved = dom_fl / (dom_ms * 1e-3) / 1e12 if dom_ms > 0 else 0.0
    all_tf = tot_fl / (tot_ms * 1e-3) / 1e12 if tot_ms > 0 else 0.0
    traffic, traffic_src = ncu_traffic(f"{w.name}.{dom}")
    roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": traffic,
                "kernel": f"tc_gemm_kernel, {dom} epilogue (largest share of device time)", "launches": dom_n,
                "flops_per_launch": dom_fl / dom_n, "avg_launch_ms": dom_ms / dom_n,
                "flops_note": "flops of the tiles computed (a symmetric product counts its upper-triangle tiles, a split "
                              "product each pass), summed over the launches and divided by their summed event time",
                "traffic_note": (f"dram__bytes_read+write per launch, ncu capture summarised in {traffic_src}"
                                 if traffic_src else "no profiler capture of this kernel at this size"),
                "peak_source": f"{peaks['source']} burst bf16 (sustained {peaks['bf16_tflops_sustained']})",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS,
                "all_contractions": {"achieved": all_tf, "frac": all_tf / peak, "launches": tot_n,
                                     "share_of_cycle": tot_ms / max(1, min(K, 4)) / (ms / K)},
                "per_epilogue": detail}

    if not g.is_main:
        D.finish(g)
        return 0

    cpu_base, parity = None, None
    if not args.no_cpu_baseline and g.world == 1:
        keep = {}
        cpu_base = cpu_oracle_sample(w, 1, keep)
        cpu_base = {k: cpu_base[k] for k in ("value", "unit", "cores", "kind", "sample")}
        parity = parity_sample(ctx, w, r0, dev, keep)
    extra = None
    if not args.no_extra and g.world == 1 and w.name == WORKLOAD:
        extra = {"c4b": heads_entry(peaks), "hadamard": hadamard_entry(peaks)}

    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": g.world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": _workload_desc(w), "tokens_per_step": cyc * w.n, "mode": "tc (bf16 operands, fp32 accumulate; "
                   "the two step products run once per cycle over its 8 queued batches; Newton-Schulz: residual product "
                   "as 1- or 3-term bf16 split on symmetric tiles, polynomial product 1 term, iterate product 2 terms "
                   "then 1)", "l2": f"inputs larger than L2: {resident_bytes / 1e6:.0f} MB "
                   f"of distinct batches resident, each read once per cycle", "replicas": g.world,
                   "input_gen_s": round(t_gen, 1)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "cpu_baseline": cpu_base, "parity_sample": parity, "extra": extra,
        "polar_update_ms": float(np.mean(upd_ms)) if upd_ms else None,
        "polar_update_ms_min": float(np.min(upd_ms)) if upd_ms else None,
        "ns_steps_used": int(st2.ns_steps_used), "orth_err": float(st2.orth_err),
        "objective_per_token_last_cycle": (j_last / n_last) if n_last else None,
        "steps_ms_per_cycle": float(np.mean(step_ms)) if step_ms else None,
        "step_only_tokens_per_s": (cyc * w.n) / (float(np.mean(step_ms)) * 1e-3) if step_ms else None,
    }
    print(json.dumps(out))
    D.finish(g)
    return 0


if __name__ == "__main__":
    sys.exit(main())
