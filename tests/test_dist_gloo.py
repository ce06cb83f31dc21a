"""The N > 1 plumbing (replicas, barrier, max-over-ranks timing, problem sharding, token-sharded statistics exchange) on
CPU with gloo, world size 2."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2605_10793_b200 import dist as D
    g = D.init(backend="gloo")
    assert g.active and g.world == 2
    D.barrier(g)
    t = D.max_over_ranks(g, 1.0 + g.rank)          # slowest rank decides
    s = D.sum_over_ranks(g, 10.0 * (g.rank + 1))
    shard = D.shard_problems(1024, g)
    odd = D.shard_problems(5, g)
    print("RESULT", g.rank, t, s, shard.start, shard.stop, odd.start, odd.stop, flush=True)
    D.barrier(g)
    D.finish(g)
""") % ROOT


SHARD_WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    from paper_2605_10793_b200 import dist as D
    from oracle import conqur_oracle as O

    class CpuCtx:                                   # stand-in for binding.Context: same calls, float64 oracle inside
        def __init__(self, d, r0): self.o = O.OpuOracle(d, r0)
        def step(self, x): self.o.step(x.numpy())
        def get_objective(self): return self.o.J, self.o.N
        def get_M(self): return torch.from_numpy(self.o.M.copy())
        def set_M(self, m, j, n): self.o.M = m.numpy().copy(); self.o.J = float(j[0]); self.o.N = int(n[0])
        def update(self): self.o.update()
        def get_R(self): return torch.from_numpy(self.o.R.copy())

    g = D.init(backend="gloo")
    d, n = 16, 90
    rng = np.random.default_rng(7)                  # the same stream on both ranks
    r0 = np.linalg.qr(rng.standard_normal((d, d)))[0]
    batches = [rng.standard_normal((n, d)) * (1.0 + 9.0 * (np.arange(d) < 2)) for _ in range(4)]
    cut = 2 * n // 3                                # uneven shards: rank 0 takes two thirds of every batch
    sh = D.TokenSharded(CpuCtx(d, r0), g)
    ref = O.OpuOracle(d, r0)
    for k, x in enumerate(batches):
        mine = x[:cut] if g.rank == 0 else x[cut:]
        if not (k == 3 and g.rank == 1):            # the last batch reaches rank 0 only
            sh.step(torch.from_numpy(mine))
        ref.step(x[:cut] if k == 3 else x)
        if k %% 2 == 1:
            j, cnt = sh.update()
            assert cnt == ref.N and abs(j - ref.J) < 1e-9 * abs(ref.J), (j, ref.J, cnt, ref.N)
            ref.update()
    err = float(np.max(np.abs(sh.ctx.get_R().numpy() - ref.R)))
    print("RESULT", g.rank, err, repr(float(sh.ctx.get_R().numpy().sum())), flush=True)
    D.barrier(g)
    D.finish(g)
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_max_time_and_shard_problems():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    rows = sorted(l.split()[1:] for o, _ in outs for l in o.splitlines() if l.startswith("RESULT"))
    assert len(rows) == 2
    for r, row in enumerate(rows):
        rank, t, s = int(row[0]), float(row[1]), float(row[2])
        assert rank == r and t == 2.0 and s == 30.0
    assert (rows[0][3:5], rows[1][3:5]) == (["0", "512"], ["512", "1024"])       # independent problems, no exchange
    assert (rows[0][5:7], rows[1][5:7]) == (["0", "3"], ["3", "5"])


def test_single_process_is_a_noop_group():
    from paper_2605_10793_b200 import dist as D
    env_backup = {k: os.environ.pop(k, None) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        g = D.init()
        assert not g.active and g.world == 1 and g.is_main
        assert D.max_over_ranks(g, 3.5) == 3.5 and list(D.shard_problems(4, g)) == [0, 1, 2, 3]
        D.barrier(g)
        D.finish(g)
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v


def test_token_sharded_update_equals_the_single_process_update():
    """Two gloo ranks, each stepping on its own (uneven) share of every batch; after each sharded update both hold the
    rotation a single process computes from all rows: M, J and N are sums over tokens, so one all-reduce of each is
    the whole exchange."""
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", SHARD_WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    rows = sorted(l.split()[1:] for o, _ in outs for l in o.splitlines() if l.startswith("RESULT"))
    assert len(rows) == 2
    assert float(rows[0][1]) < 1e-9 and float(rows[1][1]) < 1e-9       # both equal the single-process rotation
    assert rows[0][2] == rows[1][2]                                     # and each other, bit for bit
