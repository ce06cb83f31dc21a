"""conqur_objective_noalloc: the objective of a batch for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits (a runtime that owns all device memory,
a plugin in a process whose memory is pre-assigned), so they cannot hand conqur_init a workspace.  This
entry point keeps its scratch in a fixed array inside the library.  The test calls it through the C ABI
twice in a row (a large batch, then a smaller one with skipped rows, so stale scratch from the first call
would show) and checks both results against the regular conqur_step + conqur_get_objective path and against
the float64 oracle's objective and token count.
Collected last on purpose: a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _regular(x_dev, r_dev, d, dtype):
    from paper_2605_10793_b200 import binding as B
    ctx = B.Context(d=d, n_max=x_dev.shape[0], in_dtype=dtype, mode="exact")
    ctx.set_R(r_dev)
    ctx.step(x_dev)
    j, n = ctx.get_objective(check=False)
    ctx.close()
    return j, n


def test_noalloc_objective_matches_regular_path_twice_in_a_row():
    import torch
    from paper_2605_10793_b200 import binding as B
    d = 256
    w = I.scaled(I.WORKLOADS["c2"], d=d, n=3000, n_outlier=2)
    r = torch.from_numpy(I.initial_rotation(w)).cuda()
    x1 = torch.from_numpy(I.batch(w, 0)).cuda().to(torch.bfloat16)
    x2_np = I.batch(w, 1)[:777].copy()
    x2_np[5] = 0.0                      # a skipped row: the counters must not carry over from call 1
    x2_np[700, 3] = np.nan
    x2 = torch.from_numpy(x2_np).cuda()  # second call in fp32
    j_out = torch.zeros(2, dtype=torch.float64, device="cuda")
    n_out = torch.zeros(2, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    before = torch.cuda.memory_allocated()
    rc1 = B.conqur_objective_noalloc(x1.data_ptr(), B.CONQUR_BF16, x1.shape[0], d, x1.stride(0), r.data_ptr(),
                                     j_out[0:].data_ptr(), n_out[0:].data_ptr(), stream)
    rc2 = B.conqur_objective_noalloc(x2.data_ptr(), B.CONQUR_F32, x2.shape[0], d, x2.stride(0), r.data_ptr(),
                                     j_out[1:].data_ptr(), n_out[1:].data_ptr(), stream)
    assert rc1 == 0 and rc2 == 0
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before          # nothing was taken from torch's allocator either
    j1, n1 = _regular(x1, r, d, "bf16")
    j2, n2 = _regular(x2, r, d, "f32")
    got_j, got_n = j_out.cpu().numpy(), n_out.cpu().numpy()
    assert got_n[0] == n1 == 3000 and got_n[1] == n2 == 775
    assert abs(got_j[0] - j1) <= 1e-6 * abs(j1)
    assert abs(got_j[1] - j2) <= 1e-6 * abs(j2)
    # and against the definition: the oracle on the same bits (the second batch holds a zero row and a NaN row)
    r64 = r.cpu().numpy().astype(np.float64)
    o1 = O.OpuOracle(d, r64).step(x1.float().cpu().numpy().astype(np.float64))
    o2 = O.OpuOracle(d, r64).step(x2_np.astype(np.float64))
    assert got_n[0] == o1.N and got_n[1] == o2.N
    assert abs(got_j[0] - o1.J) <= 1e-6 * o1.J and abs(got_j[1] - o2.J) <= 1e-6 * o2.J


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    import torch
    from paper_2605_10793_b200 import binding as B
    x = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    r = torch.eye(64, device="cuda")
    out_j = torch.zeros(1, dtype=torch.float64, device="cuda")
    out_n = torch.zeros(1, dtype=torch.int64, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert B.conqur_objective_noalloc(x.data_ptr(), B.CONQUR_F32, 32769, 64, 64, r.data_ptr(), out_j.data_ptr(),
                                      out_n.data_ptr(), s) == -10
    assert B.conqur_objective_noalloc(x.data_ptr(), B.CONQUR_F32, 8, 8200, 8200, r.data_ptr(), out_j.data_ptr(),
                                      out_n.data_ptr(), s) == -10
    assert B.conqur_objective_noalloc(x.data_ptr(), B.CONQUR_F32, 8, 64, 64, r.data_ptr(), 0, out_n.data_ptr(), s) == -1
