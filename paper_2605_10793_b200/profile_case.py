"""A small, bounded invocation of the hot path for profiler captures.

One context, one batch through conqur_step and one conqur_update (d and n from the command line), a few
dozen launches in total, under 1 GB on the device.  Prints what it ran and the objective so that a plain
run can be checked before a capture.

  python -m paper_2605_10793_b200.profile_case [--d 4096] [--n 2048] [--mode tc] [--quant-bits 0] [--steps 1]
  python -m paper_2605_10793_b200.profile_case --op heads [--problems 592] [--n 2048]     per-head kernels (d = 128)
  python -m paper_2605_10793_b200.profile_case --op hadamard [--d 4096] [--n 16384]       Walsh-Hadamard rows, bf16
"""
from __future__ import annotations

import argparse

import numpy as np


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--n", type=int, default=2048)
    ap.add_argument("--mode", default="tc", choices=["tc", "exact"])
    ap.add_argument("--quant-bits", type=int, default=0)
    ap.add_argument("--steps", type=int, default=1, help="batches accumulated before the update")
    ap.add_argument("--ns-max-steps", type=int, default=0)
    ap.add_argument("--op", default="path", choices=["path", "heads", "hadamard"])
    ap.add_argument("--problems", type=int, default=592)
    args = ap.parse_args()

    import torch
    from paper_2605_10793_b200 import binding as B
    from paper_2605_10793_b200 import inputs as I

    if args.op == "hadamard":
        x = torch.randn(args.n, args.d, device="cuda").to(torch.bfloat16)
        y = torch.empty_like(x)
        for _ in range(3):
            B.conqur_hadamard_rows(x, out=y)
        rc = B.conqur_hadamard_status()
        print(f"profile_case hadamard n={args.n} d={args.d} bf16: status={rc} |y|max={y.float().abs().max().item():.3f}")
        return 0 if rc == 0 else 1
    if args.op == "heads":
        P, n, d = args.problems, args.n, 128
        x = (torch.randn(P * n, d, device="cuda") * (1.0 + 20.0 * (torch.arange(d, device="cuda") < 2))).to(torch.bfloat16)
        ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P)
        for _ in range(2):
            ctx.step_batched(x, n, d, n * d)
            ctx.update()
        st = ctx.get_stats()
        print(f"profile_case heads P={P} n={n}: ns_steps={st.ns_steps_used} orth={st.orth_err:.2e} status={st.status}")
        return 0 if st.status == 0 else 1

    w = I.scaled(I.WORKLOADS["c2"], d=args.d, n=args.n, quant_bits=args.quant_bits,
                 r0="hadamard" if args.d & (args.d - 1) == 0 else "qr")
    ctx = B.Context(d=args.d, n_max=args.n, in_dtype="bf16", mode=args.mode, quant_bits=args.quant_bits,
                    prior_rel=0.0 if args.steps * args.n >= 2 * args.d else 1e-2, ns_max_steps=args.ns_max_steps)
    ctx.set_R(torch.from_numpy(I.initial_rotation(w)).cuda())
    xs = [torch.from_numpy(I.batch(w, b)).cuda().to(torch.bfloat16) for b in range(args.steps)]
    torch.cuda.synchronize()
    for x in xs:
        ctx.step(x)
    j, n = ctx.get_objective()
    ctx.update()
    st = ctx.get_stats()
    print(f"profile_case d={args.d} n={args.n} mode={args.mode} steps={args.steps}: J/N={j / n:.5f} "
          f"ns_steps={st.ns_steps_used} orth={st.orth_err:.2e} status={st.status} "
          f"launches={ctx.get_profile()['total_launches']}")
    return 0 if st.status == 0 else 1


if __name__ == "__main__":
    raise SystemExit(main())
