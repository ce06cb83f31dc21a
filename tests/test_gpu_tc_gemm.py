"""The tcgen05 product in isolation (both operand orientations, plain and split precision) vs float64."""
import numpy as np
import pytest

from paper_2605_10793_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _mk(rng, rows, cols, split):
    a = rng.standard_normal((rows, cols)).astype(np.float32)
    hi = I.round_to_bf16(a)
    if not split:
        return hi.astype(np.float64), hi
    lo = I.round_to_bf16(a - hi)
    return hi.astype(np.float64) + lo.astype(np.float64), np.concatenate([hi, lo], axis=0)


def _run(m, n, k, a_mn, b_mn, split, seed=0):
    import torch
    from paper_2605_10793_b200 import binding as B
    rng = np.random.default_rng(seed)
    a_val, a_store = _mk(rng, *((k, m) if a_mn else (m, k)), split)
    b_val, b_store = _mk(rng, *((k, n) if b_mn else (n, k)), split)
    A = a_val.T if a_mn else a_val            # logical (m, k)
    Bm = b_val.T if b_mn else b_val           # logical (n, k)
    ref = A @ Bm.T
    if split:                                  # the kernel drops the lo*lo term
        a_lo = a_store[a_store.shape[0] // 2:].astype(np.float64)
        b_lo = b_store[b_store.shape[0] // 2:].astype(np.float64)
        ref = ref - (a_lo.T if a_mn else a_lo) @ (b_lo.T if b_mn else b_lo).T
    ta = torch.from_numpy(a_store).cuda().to(torch.bfloat16).contiguous()
    tb = torch.from_numpy(b_store).cuda().to(torch.bfloat16).contiguous()
    out = B.conqur_debug_gemm(ta, tb, m, n, k, a_mn, b_mn, split).cpu().numpy().astype(np.float64)
    err = np.abs(out - ref).max() / np.abs(ref).max()
    return err


def test_single_tile_k_major():
    assert _run(128, 256, 64, False, False, False) < 1e-5


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, False), (True, True)])
def test_orientations_multi_tile(a_mn, b_mn):
    assert _run(384, 512, 448, a_mn, b_mn, False, seed=1) < 2e-5


@pytest.mark.parametrize("a_mn,b_mn", [(False, True), (True, True)])
def test_ragged_m_k_and_n128(a_mn, b_mn):
    # M not a multiple of 128, K not a multiple of 64, N tiles of 128
    assert _run(200, 384, 136, a_mn, b_mn, False, seed=2) < 2e-5


@pytest.mark.parametrize("a_mn,b_mn", [(False, True), (True, True), (False, False)])
def test_split_precision_three_products(a_mn, b_mn):
    assert _run(256, 256, 320, a_mn, b_mn, True, seed=3) < 6e-6   # fp32 accumulation of 960 products


def test_many_tiles_persistent_loop():
    # more tiles than SMs: every CTA walks several tiles through both accumulator buffers
    assert _run(128 * 40, 256 * 5, 192, False, True, False, seed=4) < 2e-5


def test_bounded_wait_gives_up_and_reports_timeout():
    """A wait on a barrier nothing arrives at ends after its cycle limit with CONQUR_ERR_TIMEOUT; the kernel returns
    normally and the device keeps working (a product right after it is still correct)."""
    from paper_2605_10793_b200 import binding as B
    assert B.conqur_debug_wait_timeout(2_000_000) == -8          # about 1 ms of SM clocks
    assert "wait" in B.strerror(-8)
    test_single_tile_k_major()
