"""Guard rails on the GPU: workspace guard bands (a stand-in for a memory checker), queued (deferred) batches against
immediate ones and against the oracle, fake-quantiser bit widths other than 4, and the token-sharded wrapper driven
through the real context in a one-rank process group."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I
from tests.parity_util import TOL, assert_step, step_parity, update_parity

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torch():
    import torch
    return torch


def _dev(x, dtype="bf16"):
    torch = _torch()
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


@pytest.mark.parametrize("mode,d,batch", [("exact", 100, 1), ("tc", 256, 1), ("tc", 128, 3), ("exact", 32, 4)])
def test_guard_bands_survive_a_cycle_and_report_a_planted_overwrite(mode, d, batch):
    """Every workspace region is followed by a 256-byte band with a fixed pattern.  A whole cycle (steps with ragged
    sizes, fake-quant second pass, update) leaves all of them intact; overwriting one byte of the last band from the
    host side of the test is reported."""
    from paper_2605_10793_b200 import binding as B
    n = 333
    w = I.scaled(I.WORKLOADS["c4a"], d=d, n=n, n_outlier=2, r0="qr")
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, batch=batch, quant_bits=4, prior_rel=1e-2)
    assert ctx.cfg.debug_flags & B.CONQUR_DEBUG_CANARIES          # switched on for GPU tests by the conftest fixture
    for b in range(2):
        if batch == 1:
            ctx.step(_dev(I.batch(w, b)[: n - 7 * b]))
        else:
            xs = np.concatenate([I.batch(w, b, problem=p) for p in range(batch)], axis=0)
            ctx.step_batched(_dev(xs), n, d, n * d)
    ctx.update()
    assert ctx.get_stats().status == 0
    assert ctx.check_canaries() == 0
    nbytes = B.conqur_workspace_bytes(d, ctx.cfg)
    off = ctx._ws_ptr - ctx.workspace.data_ptr()
    saved = ctx.workspace[off + nbytes - 1].item()
    ctx.workspace[off + nbytes - 1] = (saved + 1) % 256           # the last byte of the last guard band
    assert ctx.check_canaries() == 1
    ctx.workspace[off + nbytes - 1] = saved
    assert ctx.check_canaries() == 0
    B.DEBUG_CANARIES = False                                       # a context created without the flag has no bands to check
    try:
        plain = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, batch=batch)
    finally:
        B.DEBUG_CANARIES = True
    assert B.load().conqur_debug_check_canaries(plain.h) == -1


@pytest.mark.parametrize("quant", [(0, "sym", 1.0), (4, "zp", 0.9)])
def test_queued_batches_equal_immediate_ones_and_the_oracle(quant):
    """A context that queues its batches (defer_batches = cadence) and runs the two products once over all queued
    rows gives the statistics of a context that runs them per batch (same sign decisions, same token count; sums
    differ by fp32 summation order only), matches the oracle on the pooled rows, and flushes whenever something reads
    or replaces the statistics."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    bits, qmode, clip = quant
    d, n, K = 512, 600, 4
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    r0 = I.initial_rotation(w)
    xs = [I.batch(w, b)[: n - 50 * (b % 2)] for b in range(K + 1)]            # ragged batch sizes
    xs[1] = xs[1].copy(); xs[1][5] = 0.0                                       # a skipped row in a queued batch
    kw = dict(d=d, n_max=n, in_dtype="bf16", mode="tc", quant_bits=bits, quant_mode=qmode, clip_ratio=clip)
    now, later = B.Context(**kw), B.Context(defer_batches=K, **kw)
    for c in (now, later):
        c.set_R(_dev(r0, "f32"))
    signs_now = []
    for x in xs[:K]:
        now.step(_dev(x))
        signs_now.append(now.debug_get_signs(x.shape[0]).cpu().numpy())
        later.step(_dev(x))
    rows = sum(x.shape[0] for x in xs[:K])
    (j1, n1), (j2, n2) = now.get_objective(), later.get_objective()
    assert n1 == n2 == rows - 1 and abs(j1 - j2) <= 1e-6 * abs(j1)
    s_later = later.debug_get_signs(rows).cpu().numpy()
    assert np.array_equal(s_later, np.concatenate(signs_now, axis=0))
    m1, m2 = now.get_M().cpu().numpy().astype(np.float64), later.get_M().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(m1 - m2) <= 1e-5 * np.linalg.norm(m1)
    x_all = np.concatenate(xs[:K], axis=0).astype(np.float64)
    rep = step_parity(x_all, r0.astype(np.float64), s_later, m2, j2, n2, "tc", bits, quant_mode=qmode, clip_ratio=clip)
    assert_step(rep, "tc", 2e-2)
    # a partial queue is flushed by the update; the next cycle starts from an empty queue
    later.update(); now.update()
    assert later.get_stats().status == 0
    rep = update_parity(m2, later.get_R().cpu().numpy().astype(np.float64))
    assert rep["orth"] <= TOL["tc"]["orth"] and rep["gap"] <= TOL["tc"]["gap"], rep
    later.step(_dev(xs[K]))
    later.set_R(later.get_R())                                                 # replacing R flushes what was queued under it
    j3, n3 = later.get_objective()
    ref = O.OpuOracle(d, later.get_R().cpu().numpy().astype(np.float64), quant_bits=bits, quant_mode=qmode, clip_ratio=clip)
    ref.step(xs[K].astype(np.float64))
    assert n3 == ref.N and abs(j3 - ref.J) <= TOL["tc"]["J"] * ref.J


@pytest.mark.parametrize("mode,d,batch,defer", [("exact", 96, 1, 0), ("tc", 256, 1, 3), ("tc", 128, 5, 0), ("exact", 32, 3, 0)])
def test_asynchronous_objective_read(mode, d, batch, defer):
    """conqur_get_objective_async leaves (J, N) as of its point in the stream in page-locked host arrays without
    stopping the stream: the values equal the synchronous read taken at the same point, also when an update that resets
    the sums is enqueued behind it (the per-head tensor-core case forms J from M on the way)."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    n = 300
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2, r0="qr")
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, batch=batch, defer_batches=defer)
    jh = torch.zeros(batch, dtype=torch.float64).pin_memory()
    nh = torch.zeros(batch, dtype=torch.int64).pin_memory()
    for cycle in range(2):
        for b in range(2):
            if batch == 1:
                ctx.step(_dev(I.batch(w, 2 * cycle + b)))
            else:
                x = np.stack([I.batch(w, 10 * p + 2 * cycle + b) for p in range(batch)])
                ctx.step_batched(_dev(x.reshape(batch * n, d)), n, d, n * d)
        j_sync, n_sync = ctx.get_objective()
        ctx.get_objective_async(jh, nh)
        ctx.update()                                   # enqueued behind the read: resets the sums on the device
        ctx.stream.synchronize()
        assert np.array_equal(nh.numpy(), np.atleast_1d(n_sync)) and np.all(nh.numpy() == 2 * n)
        assert np.array_equal(jh.numpy(), np.atleast_1d(j_sync)) and np.all(jh.numpy() > 0)
        j0, n0 = ctx.get_objective()
        assert np.all(np.atleast_1d(n0) == 0) and np.all(np.atleast_1d(j0) == 0.0)
        st = ctx.get_stats()
        assert st.status == 0 and abs(st.last_J - float(np.sum(jh.numpy()))) <= 1e-9 * st.last_J


@pytest.mark.parametrize("mode", ["exact", "tc"])
@pytest.mark.parametrize("bits", [2, 3, 8])
@pytest.mark.parametrize("qmode,clip", [("sym", 1.0), ("zp", 0.9)])
def test_fake_quant_bit_widths(mode, bits, qmode, clip):
    """Appendix B's quantisers at 2, 3 and 8 bits (4 is covered everywhere else): objective, tie-aware
    cross-covariance and the band of every differing decision, single problem and per-head problems."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    d, n = 256, 700
    w = I.scaled(I.WORKLOADS["c4a"], d=d, n=n, n_outlier=2)
    x = I.batch(w, 0)
    r0 = I.initial_rotation(w)
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, quant_bits=bits, quant_mode=qmode, clip_ratio=clip)
    ctx.set_R(_dev(r0, "f32"))
    ctx.step(_dev(x))
    j, nn = ctx.get_objective()
    m = ctx.get_M().cpu().numpy().astype(np.float64)
    s = ctx.debug_get_signs(n).cpu().numpy()
    rep = step_parity(x.astype(np.float64), r0.astype(np.float64), s, m, j, nn, mode, bits, quant_mode=qmode, clip_ratio=clip)
    if mode == "exact" and qmode == "zp":
        rep["J_rel"] = rep["J_rel"] / 10.0          # a tie in the integer zero-point moves a clamped code by one level
    assert_step(rep, mode, 2e-2 if mode == "tc" else 1e-3)
    # per-head problems through the batched kernels
    P, n2, dh = 3, 300, 128
    wb = I.scaled(I.WORKLOADS["c4b"], n=n2, problems=P)
    xs = [I.batch(wb, 0, problem=p) for p in range(P)]
    rh = np.stack([I.initial_rotation(wb, p) for p in range(P)])
    cb = B.Context(d=dh, n_max=n2, in_dtype="bf16", mode=mode, batch=P, quant_bits=bits, quant_mode=qmode, clip_ratio=clip)
    cb.set_R(_dev(rh, "f32"))
    signs = torch.zeros((P, n2, dh), dtype=torch.int8, device="cuda")
    if mode == "tc":
        cb.debug_capture_signs(signs)
    cb.step_batched(_dev(np.concatenate(xs, axis=0)), n2, dh, n2 * dh)
    if mode == "exact":
        signs = cb.debug_get_signs(n2, problems=P)
    js, ns = cb.get_objective()
    ms = cb.get_M().cpu().numpy().astype(np.float64)
    for p in range(P):
        rep = step_parity(xs[p].astype(np.float64), rh[p].astype(np.float64), signs[p].cpu().numpy(), ms[p], js[p], ns[p], mode,
                          bits, quant_mode=qmode, clip_ratio=clip)
        if mode == "exact" and qmode == "zp":
            rep["J_rel"] = rep["J_rel"] / 10.0
        assert_step(rep, mode, 2e-2 if mode == "tc" else 1e-3)


def test_single_cta_kernels_on_a_device_that_would_use_pairs():
    """The 128-row single-CTA variants of the tensor-core product (used where CTA pairs cannot be co-scheduled)."""
    from paper_2605_10793_b200 import binding as B
    d, n = 512, 700
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    r0 = I.initial_rotation(w)
    x = I.batch(w, 0)
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", debug_flags=B.CONQUR_DEBUG_SINGLE_CTA | B.CONQUR_DEBUG_NO_GRAPH)
    ctx.set_R(_dev(r0, "f32"))
    for cyc in range(2):
        r = ctx.get_R().cpu().numpy().astype(np.float64)
        ctx.step(_dev(x))
        j, nn = ctx.get_objective()
        m = ctx.get_M().cpu().numpy().astype(np.float64)
        s = ctx.debug_get_signs(n).cpu().numpy()
        assert_step(step_parity(x.astype(np.float64), r, s, m, j, nn, "tc"), "tc", 2e-2)
        ctx.update()
        assert ctx.get_stats().status == 0
        rep = update_parity(m, ctx.get_R().cpu().numpy().astype(np.float64))
        assert rep["orth"] <= TOL["tc"]["orth"] and rep["gap"] <= TOL["tc"]["gap"], rep


SHARD_WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    from paper_2605_10793_b200 import binding as B, dist as D, inputs as I
    from oracle import conqur_oracle as O
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%%d" %% int(sys.argv[1]), rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    g = D.Group(0, 0, 1, True)
    d, n = 256, 1000
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    r0 = I.initial_rotation(w)
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc")
    ctx.set_R(torch.from_numpy(r0).cuda())
    sh = D.TokenSharded(ctx, g)
    ref = O.OpuOracle(d, r0.astype(np.float64))
    for b in range(3):
        x = I.batch(w, b)
        sh.step(torch.from_numpy(x).cuda().to(torch.bfloat16))
        ref.step(x.astype(np.float64))
    m = ctx.get_M().cpu().numpy().astype(np.float64)
    j, cnt = sh.update()                      # get_M -> all-reduce -> set_M -> update, on the real context
    st = ctx.get_stats()
    r = ctx.get_R().cpu().numpy().astype(np.float64)
    r_ref, sig = O.polar_svd(m)
    gap = 1.0 - np.sum(r * m) / sig.sum()
    orth = np.max(np.abs(r.T @ r - np.eye(d)))
    print("RESULT", st.status, cnt == ref.N, abs(j - ref.J) / ref.J, gap, orth, st.last_N, flush=True)
    dist.destroy_process_group()
""") % ROOT


def test_token_sharded_wrapper_over_the_real_context_one_rank():
    """dist.TokenSharded on binding.Context with an initialised (one-rank, NCCL) process group: the statistics leave
    through conqur_get_M, pass the all-reduce, re-enter through conqur_set_M, and the update on them matches the
    oracle's polar factor."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, NCCL_NVLS_ENABLE="0")
    p = subprocess.run([sys.executable, "-c", SHARD_WORKER, str(port)], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    row = [l.split()[1:] for l in p.stdout.splitlines() if l.startswith("RESULT")][0]
    assert int(row[0]) == 0 and row[1] == "True"
    assert float(row[2]) <= TOL["tc"]["J"] and float(row[3]) <= TOL["tc"]["gap"] and float(row[4]) <= TOL["tc"]["orth"]
    assert int(row[5]) == 3000


def test_looped_update_graph_equals_direct_launches_bit_for_bit():
    """After a context's first update the launch sequence is replayed from a captured graph whose middle is a
    device-side loop over Newton-Schulz steps; CONQUR_DEBUG_NO_GRAPH enqueues every launch directly.  Same kernels,
    same order, same data: rotations, statistics and step counts are identical over several cycles."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    d, n = 512, 1024
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=n, n_outlier=2)
    xs = [_dev(I.batch(w, b)) for b in range(6)]
    out = []
    for flags in (0, B.CONQUR_DEBUG_NO_GRAPH):
        ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", defer_batches=2, debug_flags=flags)
        ctx.set_R(_dev(I.initial_rotation(w), "f32"))
        trace = []
        for cyc in range(5):
            ctx.step(xs[cyc % 6]); ctx.step(xs[(cyc + 1) % 6])
            ctx.update()
            st = ctx.get_stats()
            assert st.status == 0
            trace.append((ctx.get_R().clone(), int(st.ns_steps_used), int(st.ns_lift_plan), st.last_J))
        out.append(trace)
    for a, b in zip(*out):
        assert torch.equal(a[0], b[0]) and a[1:] == b[1:]
    launches = ctx.get_profile()["total_launches"]
    assert launches > 0


def test_per_head_step_timeline_hook():
    """conqur_debug_trace_heads: thread block 0 stamps its first tiles; the events of a tile come in the order the
    pipeline imposes (copy issued < first product < epilogue done < second product) and nothing is written once the
    hook is switched off."""
    from paper_2605_10793_b200 import binding as B
    torch = _torch()
    P, n, d = 148, 512, 128                              # one problem per thread block, four tiles each
    x = (torch.randn(P * n, d, device="cuda") * (1.0 + 20.0 * (torch.arange(d, device="cuda") < 2))).to(torch.bfloat16)
    ctx = B.Context(d=d, n_max=n, in_dtype="bf16", mode="tc", batch=P)
    trace = torch.zeros(96 * 16, dtype=torch.int64, device="cuda")
    ctx.debug_trace_heads(trace)
    ctx.step_batched(x, n, d, n * d)
    ctx.debug_trace_heads(None)
    t = trace.cpu().numpy().reshape(96, 16)
    tiles = n // 128
    used = t[:tiles]
    assert (used[:, [0, 1, 2, 5, 9]] > 0).all()
    assert (used[:, 0] < used[:, 1]).all() and (used[:, 1] < used[:, 9]).all() and (used[:, 9] < used[:, 2]).all()
    assert not t[tiles:].any()                                       # block 0 worked on one problem only
    trace.zero_()
    ctx.step_batched(x, n, d, n * d)
    torch.cuda.synchronize()
    assert not trace.any().item()
    assert ctx.get_stats().status == 0
