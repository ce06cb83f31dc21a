"""GPU parity of Algorithm 1's site scheduling: the shared R_1 context fed by every block's two residual-stream
sites, one batched context of all per-head problems fed block by block from head-interleaved o_proj inputs and
updated once per mini-batch, against the oracle's Algorithm-1 composition (which updates each block's heads
inside the loop over blocks, as the paper writes it).  Teacher-forced per mini-batch: the oracle starts each mini-batch from the library's
current rotations, so differences are that mini-batch's own arithmetic."""
import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I
from tests.parity_util import TOL, assert_step, log_parity, step_parity, unit_roundoff, update_parity

pytestmark = pytest.mark.gpu

# flipped-sign fraction allowed (every flipped sign must also lie inside the rounding band)
FLIP_MAX = {"exact": 1e-3, "tc": 2e-2}


def _torch():
    import torch
    return torch


@pytest.mark.parametrize("mode,quant", [("exact", (0, "sym", 1.0)), ("tc", (0, "sym", 1.0)), ("tc", (4, "zp", 0.9))])
def test_algorithm1_small_model_against_the_oracle(mode, quant):
    torch = _torch()
    from paper_2605_10793_b200 import algorithm1 as A1
    a = I.SITE_MODELS["a1_small"]
    T = TOL[mode]
    bits, qmode, clip = quant
    cal = A1.Calibrator(a.d, a.n_heads, a.d_head, a.n_layers, a.n, in_dtype="bf16", mode=mode, quant_bits=bits,
                        quant_mode=qmode, clip_ratio=clip, record="full")
    r1, r2 = I.site_initial_rotations(a)
    cal.set_rotations(torch.from_numpy(r1).cuda(), torch.from_numpy(r2).cuda())
    for mb in range(a.n_minibatches):
        g1, g2 = cal.rotations()
        g1, g2 = g1.cpu().numpy().astype(np.float64), g2.cpu().numpy().astype(np.float64)
        sites = [I.site_activations(a, mb, l) for l in range(a.n_layers)]
        for l, s in enumerate(sites):
            dev = {k: torch.from_numpy(v).cuda().to(torch.bfloat16) for k, v in s.items()}
            cal.collect(l, dev["attn"], dev["mlp"], dev["o"])
        cal.end_minibatch()
        assert cal.ctx1.get_stats().status == 0
        sites64 = [{k: v.astype(np.float64) for k, v in s.items()} for s in sites]
        _, _, log = O.run_algorithm1(a.d, a.n_heads, a.d_head, a.n_layers, [sites64], g1, g2, quant_bits=bits,
                                     quant_mode=qmode, clip_ratio=clip)
        ref, got = log[0], cal.log[mb]
        # the shared rotation's problem: all 2L sites pooled
        assert got["N1"] == ref["N1"] == 2 * a.n_layers * a.n
        assert abs(got["J1"] - ref["J1"]) / ref["J1"] <= T["J"]
        # its cross-covariance, tie-aware: the oracle pools the 2L sites with the sign decisions the library took,
        # and every decision that differs from the oracle's own lies inside the rounding band
        orc = O.OpuOracle(a.d, g1, bits, 0.0, qmode, clip)
        ta = O.OpuOracle(a.d, g1, bits, 0.0, qmode, clip)
        flips = total = 0
        for l, s in enumerate(sites64):
            for site in ("attn", "mlp"):
                s_gpu = got["signs"][(site, l)].astype(np.float64)
                orc.step(s[site])
                ta.step(s[site], signs_override=s_gpu)
                diff = s_gpu != orc.last_S
                flips += int(diff.sum()); total += diff.size
                if bits == 0:
                    xt, _ = O.normalise_rows(s[site])
                    band = 6.0 * unit_roundoff(mode, a.d) * np.sqrt((xt * xt) @ (g1 * g1))
                    assert not (diff & (np.abs(orc.last_Y) > band)).any()
        m1 = got["M1"].astype(np.float64)
        rep1 = {"M_rel_tie_aware": float(np.linalg.norm(m1 - ta.M) / np.linalg.norm(ta.M)),
                "M_rel_raw": float(np.linalg.norm(m1 - orc.M) / np.linalg.norm(orc.M)), "flip_frac": flips / total,
                "J_rel": abs(got["J1"] - ref["J1"]) / ref["J1"]}
        log_parity("a1_small", mode, f"R_1 pooled problem, mini-batch {mb}, quant {quant}", rep1)
        assert rep1["M_rel_tie_aware"] <= T["M"] and rep1["flip_frac"] < FLIP_MAX[mode], rep1
        n1, n2 = cal.rotations()
        n1, n2 = n1.cpu().numpy().astype(np.float64), n2.cpu().numpy().astype(np.float64)
        rep = update_parity(m1, n1)
        assert rep["orth"] <= T["orth"] and rep["gap"] <= T["gap"], rep
        # every head of every block: its own problem, updated inside the loop over blocks
        for l in range(a.n_layers):
            for h in range(a.n_heads):
                assert got["N2"][l, h] == ref["N2"][l, h] == a.n
                assert abs(got["J2"][l, h] - ref["J2"][l, h]) / ref["J2"][l, h] <= T["J"], (l, h)
                mh = got["M2"][l, h].astype(np.float64)
                srep = step_parity(sites64[l]["o"][:, h * a.d_head:(h + 1) * a.d_head], g2[l, h], got["signs"][("o", l)][h], mh,
                                   got["J2"][l, h], got["N2"][l, h], mode, bits, quant_mode=qmode, clip_ratio=clip)
                assert_step(srep, mode, FLIP_MAX[mode])
                rep = update_parity(mh, n2[l, h])
                assert rep["orth"] <= T["orth"] and rep["gap"] <= T["gap"], (l, h, rep)
    cal.close()


def test_algorithm1_free_running_matches_the_oracle_chain():
    """No teacher forcing: both sides run both mini-batches from the same initial rotations (exact mode); the final
    rotations agree to the accuracy the conditioning of the polar factor allows."""
    torch = _torch()
    from paper_2605_10793_b200 import algorithm1 as A1
    a = I.SITE_MODELS["a1_small"]
    cal = A1.Calibrator(a.d, a.n_heads, a.d_head, a.n_layers, a.n, in_dtype="bf16", mode="exact")
    r1, r2 = I.site_initial_rotations(a)
    cal.set_rotations(torch.from_numpy(r1).cuda(), torch.from_numpy(r2).cuda())
    mbs = []
    for mb in range(a.n_minibatches):
        sites = [I.site_activations(a, mb, l) for l in range(a.n_layers)]
        mbs.append([{k: v.astype(np.float64) for k, v in s.items()} for s in sites])
        for l, s in enumerate(sites):
            cal.collect(l, *(torch.from_numpy(s[k]).cuda().to(torch.bfloat16) for k in ("attn", "mlp", "o")))
        cal.end_minibatch()
    o1, o2, _ = O.run_algorithm1(a.d, a.n_heads, a.d_head, a.n_layers, mbs, r1.astype(np.float64), r2.astype(np.float64))
    g1, g2 = cal.rotations()
    g1, g2 = g1.cpu().numpy().astype(np.float64), g2.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(g1 - o1) / np.sqrt(a.d) <= 5e-3
    assert np.linalg.norm(g2 - o2) / np.sqrt(g2.size / a.d_head) <= 5e-3
    cal.close()


@pytest.mark.parametrize("mode", ["exact", "tc"])
def test_problem_ranges_of_a_batched_context(mode):
    """conqur_step_batched_range: feeding a context's problems range by range (in any order, ranges of different
    sizes, stacked and head-interleaved inputs) gives what one conqur_step_batched over all problems gives (up to the
    fp32 rounding of a different grouping of the token tiles: a call on few problems splits each problem's tokens over
    several CTAs); an update with an unfed problem is refused."""
    torch = _torch()
    from paper_2605_10793_b200 import binding as B
    w = I.scaled(I.WORKLOADS["c4b"], n=300, problems=7)
    P, d, n = 7, w.d, w.n
    xs = [I.batch(w, 0, problem=p) for p in range(P)]
    r0 = torch.from_numpy(np.stack([I.initial_rotation(w, p) for p in range(P)])).cuda()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(torch.bfloat16)
    whole = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, batch=P)
    whole.set_R(r0)
    whole.step_batched(dev(np.concatenate(xs, axis=1)), n, P * d, d)
    jw, nw = whole.get_objective()
    mw = whole.get_M().cpu().numpy()
    parts = B.Context(d=d, n_max=n, in_dtype="bf16", mode=mode, batch=P)
    parts.set_R(r0)
    parts.step_batched_range(dev(np.concatenate(xs[4:7], axis=1)), n, 3 * d, d, 4, 3)       # interleaved, last three
    assert B.conqur_update(parts.h) == -4                                                   # problems 0..3 have no rows yet
    parts.step_batched_range(dev(np.concatenate(xs[0:3], axis=0)), n, d, n * d, 0, 3)       # stacked, first three
    parts.step_batched_range(dev(xs[3]), n, d, 0, 3, 1)                                     # a single problem
    jp, npp = parts.get_objective()
    assert np.array_equal(nw, npp) and np.allclose(jw, jp, rtol=1e-12, atol=0)
    mp = parts.get_M().cpu().numpy()
    assert np.max(np.abs(mw - mp)) <= 1e-5 * np.max(np.abs(mw))
    whole.update()
    parts.update()
    assert np.max(np.abs(whole.get_R().cpu().numpy() - parts.get_R().cpu().numpy())) <= 1e-3
    lib = B.load()
    x = dev(xs[0])
    assert lib.conqur_step_batched_range(parts.h, x.data_ptr(), n, d, n * d, 6, 2) == -1    # past the last problem
    assert lib.conqur_step_batched_range(parts.h, x.data_ptr(), n, d, n * d, -1, 1) == -1
    assert lib.conqur_step_batched_range(parts.h, x.data_ptr(), n, d, n * d, 0, 0) == -1
