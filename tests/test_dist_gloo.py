"""The N > 1 plumbing (replicas, barrier, max-over-ranks timing, problem sharding) on CPU with gloo, world size 2."""
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
