"""GPU parity of the Appendix-A pieces around the calibration path: weight folding and the Walsh-Hadamard row
transform, through the C ABI, against the float64 oracle."""
import numpy as np
import pytest

from oracle import conqur_oracle as O
from paper_2605_10793_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _B():
    from paper_2605_10793_b200 import binding as B
    return B


def _orth32(seed, d):
    q, r = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, d)))
    return (q * np.sign(np.diag(r))[None, :]).astype(np.float32)


# ------------------------------------------------------------------------------------------ Walsh-Hadamard
@pytest.mark.parametrize("d", [4, 8, 32, 64, 128, 256, 512, 1024, 2048, 4096, 8192])
@pytest.mark.parametrize("io", [("f32", "f32"), ("bf16", "bf16"), ("bf16", "f32"), ("f32", "bf16")])
def test_hadamard_rows_match_the_matrix_definition(d, io):
    torch = _torch()
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}
    n = 37 if d >= 1024 else 523                       # ragged against the rows one CTA covers
    rng = np.random.default_rng(d)
    x = rng.standard_t(3.0, size=(n, d)).astype(np.float32)
    x[:, 1] *= 50.0                                    # an outlier channel, as in the activations these transforms see
    if io[0] == "bf16":
        x = I.round_to_bf16(x)
    xd = torch.from_numpy(x).cuda().to(tdt[io[0]])
    y = _B().conqur_hadamard_rows(xd, out_dtype=tdt[io[1]])
    assert y.dtype == tdt[io[1]] and y.shape == (n, d)
    ref = O.hadamard_rows(x.astype(np.float64))
    got = y.float().cpu().numpy().astype(np.float64)
    # log2(d) fp32 butterfly levels: |err| <= log2(d) 2^-24 ||x||_1 / sqrt(d) <= log2(d) 2^-24 ||x||_2; bf16 output adds 2^-9 |y|
    bound = np.log2(d) * 2.0 ** -24 * np.linalg.norm(x.astype(np.float64), axis=1, keepdims=True)
    if io[1] == "bf16":
        bound = bound + 2.0 ** -8 * np.abs(ref)
    assert (np.abs(got - ref) <= bound + 1e-30).all(), float(np.max(np.abs(got - ref) / (bound + 1e-30)))
    assert _B().conqur_hadamard_status() == 0


@pytest.mark.parametrize("d,n", [(128, 40000), (4096, 3000), (8192, 700)])
def test_hadamard_many_blocks_per_cta(d, n):
    """More blocks than resident CTAs, so every CTA walks several blocks through its ring of stages; rows with an odd
    16-byte-unaligned stride take the plain-load kernel and must agree bit for bit."""
    torch = _torch()
    B = _B()
    x = torch.randn(n, d, device="cuda")
    y = B.conqur_hadamard_rows(x)
    assert B.conqur_hadamard_status() == 0
    sel = np.random.default_rng(0).choice(n, size=64, replace=False)
    ref = O.hadamard_rows(x[sel].cpu().numpy().astype(np.float64))
    bound = np.log2(d) * 2.0 ** -24 * np.linalg.norm(x[sel].cpu().numpy().astype(np.float64), axis=1, keepdims=True)
    assert (np.abs(y[sel].cpu().numpy() - ref) <= bound).all()
    # involution over the whole array (every block of every CTA)
    z = B.conqur_hadamard_rows(y)
    assert torch.allclose(z, x, atol=1e-4)
    xb = x.to(torch.bfloat16)
    view = torch.zeros(n, d + 8, dtype=torch.bfloat16, device="cuda")
    v4 = view[:, 4:4 + d]                                        # bf16 rows 8 bytes off a 16-byte boundary: plain-load kernel
    v4.copy_(xb)
    assert v4.data_ptr() % 16 == 8
    y_tc = B.conqur_hadamard_rows(xb, out_dtype=torch.float32)           # contiguous bf16: tensor-core kernel
    y_bulk = B.conqur_hadamard_rows(xb, out_dtype=torch.float32, cuda_cores_only=True)   # ... and the bulk-copy CUDA-core kernel
    assert torch.equal(B.conqur_hadamard_rows(v4, out_dtype=torch.float32), y_bulk)
    assert B.conqur_hadamard_status() == 0
    tol = float(np.log2(d)) * 2.0 ** -23 * torch.linalg.norm(xb.float(), dim=1, keepdim=True)
    assert ((y_tc - y_bulk).abs() <= tol).all()


def test_hadamard_strides_in_place_empty_and_argument_errors():
    torch = _torch()
    B = _B()
    d, n = 512, 100
    x = torch.randn(n, d + 64, device="cuda")
    view = x[:, 32:32 + d]                              # row stride d + 64, offset 128 bytes
    out = torch.zeros(n, d + 8, device="cuda")
    B.conqur_hadamard_rows(view, out=out[:, :d])
    ref = O.hadamard_rows(view.cpu().numpy().astype(np.float64))
    assert np.allclose(out[:, :d].cpu().numpy(), ref, atol=2e-5)
    assert not out[:, d:].any().item()                  # nothing written past the row
    # in place, and twice = identity (H/sqrt(d) is its own inverse)
    z = view.clone().contiguous()
    z0 = z.clone()
    B.conqur_hadamard_rows(z, out=z)
    assert np.allclose(z.cpu().numpy(), ref, atol=2e-5)
    B.conqur_hadamard_rows(z, out=z)
    assert torch.allclose(z, z0, atol=2e-5)
    # in place on contiguous bf16 rows (the tensor-core kernel): same result as out of place
    zb = torch.randn(3000, 1024, device="cuda").to(torch.bfloat16)
    want = B.conqur_hadamard_rows(zb)
    B.conqur_hadamard_rows(zb, out=zb)
    assert torch.equal(zb, want) and B.conqur_hadamard_status() == 0
    # empty input is a no-op; bad sizes are refused
    e = torch.empty(0, d, device="cuda")
    assert B.conqur_hadamard_rows(e).shape == (0, d)
    lib = B.load()
    s = torch.cuda.current_stream().cuda_stream
    good = torch.zeros(4, 96, device="cuda")
    assert lib.conqur_hadamard_rows(good.data_ptr(), 0, 4, 96, 96, good.data_ptr(), 0, 96, 0, s) == -1    # not a power of two
    assert lib.conqur_hadamard_rows(good.data_ptr(), 0, 4, 16384, 16384, good.data_ptr(), 0, 16384, 0, s) == -1
    assert lib.conqur_hadamard_rows(good.data_ptr(), 0, 4, 64, 32, good.data_ptr(), 0, 64, 0, s) == -1    # stride < d
    assert lib.conqur_hadamard_rows(good.data_ptr() + 4, 0, 4, 64, 96, good.data_ptr(), 0, 96, 0, s) == -1  # misaligned
    assert lib.conqur_hadamard_rows(good.data_ptr(), 7, 4, 64, 96, good.data_ptr(), 0, 96, 0, s) == -1
    assert not good.any().item()


def test_hadamard_matches_the_initial_rotation_recipe_at_headline_width():
    """x (H diag(s)) / sqrt(d), the randomised Hadamard R_0 of the headline workload, from the butterfly kernel:
    transform, then flip the signed columns."""
    torch = _torch()
    w = I.WORKLOADS["c2"]
    r0 = I.initial_rotation(w).astype(np.float64)
    x = I.batch(I.scaled(w, n=256), 0)
    y = _B().conqur_hadamard_rows(torch.from_numpy(x).cuda()).cpu().numpy().astype(np.float64)
    s = np.sign(r0[0])                                  # row 0 of H is all ones: the column signs
    ref = x.astype(np.float64) @ r0
    bound = np.log2(w.d) * 2.0 ** -24 * np.linalg.norm(x.astype(np.float64), axis=1, keepdims=True)
    assert (np.abs(y * s[None, :] - ref) <= bound).all()


# ------------------------------------------------------------------------------------------ weight folding
FOLD_TOL = {"exact": 2e-6, "tc": 2e-5}


def _fold_check(w, r_blocks, side, mode):
    torch = _torch()
    got = _B().conqur_fold_weight(torch.from_numpy(w).cuda(), torch.from_numpy(r_blocks).cuda(), side, mode)
    ref = O.fold_weight(w.astype(np.float64), r_blocks.astype(np.float64), side)
    got = got.cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    # element-wise against the size of the terms of each inner product
    rfull = np.abs(O.block_diag_rotation(r_blocks.astype(np.float64)))
    mag = np.abs(w.astype(np.float64)) @ rfull if side == "input" else rfull.T @ np.abs(w.astype(np.float64))
    elem = np.max(np.abs(got - ref) / (mag + 1e-300))
    return rel, elem


@pytest.mark.parametrize("mode", ["exact", "tc"])
@pytest.mark.parametrize("side,rows,cols", [("input", 384, 256), ("input", 136, 256), ("output", 256, 160),
                                            ("output", 256, 1024), ("input", 2048, 1024), ("output", 1024, 1536)])
def test_fold_full_rotation(mode, side, rows, cols):
    d = cols if side == "input" else rows
    w = I.random_weight(rows * 7 + cols, rows, cols)
    w[:, 0] *= 30.0
    r = _orth32(d, d)
    rel, elem = _fold_check(w, r, side, mode)
    assert rel <= FOLD_TOL[mode], (rel, elem)
    assert elem <= 4 * FOLD_TOL[mode], (rel, elem)


@pytest.mark.parametrize("mode", ["exact", "tc"])
@pytest.mark.parametrize("side,rows,cols,nh,dh", [("input", 200, 384, 3, 128), ("output", 384, 200, 3, 128),
                                                  ("input", 100, 96, 3, 32), ("output", 160, 77, 5, 32)])
def test_fold_block_diagonal_rotation(mode, side, rows, cols, nh, dh):
    w = I.random_weight(rows * 3 + cols, rows, cols)
    blocks = np.stack([_orth32(50 + h, dh) for h in range(nh)])
    rel, elem = _fold_check(w, blocks, side, mode)
    assert rel <= FOLD_TOL["exact"] and elem <= 4 * FOLD_TOL["exact"], (rel, elem)      # fp32 product in either mode


def test_fold_strided_weight_and_refusals():
    torch = _torch()
    B = _B()
    d, rows = 256, 128
    big = torch.from_numpy(I.random_weight(5, rows, d + 64)).cuda()
    w = big[:, 64:]                                      # row stride d + 64
    r = torch.from_numpy(_orth32(9, d)).cuda()
    ref = O.fold_weight(w.cpu().numpy().astype(np.float64), r.cpu().numpy().astype(np.float64), "input")
    for mode in ("exact", "tc"):
        got = B.conqur_fold_weight(w, r, "input", mode).cpu().numpy()
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= FOLD_TOL[mode]
    lib = B.load()
    s = torch.cuda.current_stream().cuda_stream
    out = torch.zeros(rows, d, device="cuda")
    scratch = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    wc = w.contiguous()
    args = lambda **k: [k.get("w", wc).data_ptr(), k.get("ldw", d), k.get("rows", rows), k.get("cols", d), r.data_ptr(),
                        k.get("block", d), k.get("side", 0), k.get("mode", 1), k.get("out", out).data_ptr(), k.get("ldo", d),
                        scratch.data_ptr(), k.get("sb", scratch.numel()), s]
    assert lib.conqur_fold_weight(*args(block=96)) == -1                 # folded dimension not a multiple of the block
    assert lib.conqur_fold_weight(*args(side=2)) == -1
    assert lib.conqur_fold_weight(*args(out=wc)) == -1                   # in place
    assert lib.conqur_fold_weight(*args(sb=1024)) == -2                  # scratch too small
    assert lib.conqur_fold_weight(*args(rows=100)) == -10               # tensor-core route needs rows % 8 == 0
    assert B.conqur_fold_scratch_bytes(rows, d, 96, 0, 1) == -1
    assert not out.any().item()


def test_folded_block_reproduces_the_rotated_outputs():
    """Appendix A end to end on the device: fold R_1 and per-head R_2 into a block's projections, then the value ->
    output chain and the MLP chain on rotated inputs give the rotated outputs of the original weights."""
    torch = _torch()
    from paper_2605_10793_b200 import algorithm1 as A1
    d, nh, dh, dff, t = 256, 2, 128, 384, 64
    names = {"q": (d, d), "k": (d, d), "v": (nh * dh, d), "o": (d, nh * dh), "up": (dff, d), "gate": (dff, d), "down": (d, dff)}
    w = {k: I.random_weight(i, *shape) for i, (k, shape) in enumerate(names.items())}
    r1 = _orth32(1, d)
    r2 = np.stack([_orth32(10 + h, dh) for h in range(nh)])
    for mode in ("exact", "tc"):
        f = A1.fold_block({k: torch.from_numpy(v).cuda() for k, v in w.items()}, torch.from_numpy(r1).cuda(),
                          torch.from_numpy(r2).cuda(), mode)
        f = {k: v.cpu().numpy().astype(np.float64) for k, v in f.items()}
        x = np.random.default_rng(3).standard_normal((t, d))
        w64 = {k: v.astype(np.float64) for k, v in w.items()}
        r1d, r2d = r1.astype(np.float64), O.block_diag_rotation(r2.astype(np.float64))
        xr = x @ r1d
        tol = 50 * FOLD_TOL[mode]
        for k in ("q", "k", "up", "gate"):
            assert np.allclose(xr @ f[k].T, x @ w64[k].T, atol=tol), k
        v_rot = xr @ f["v"].T
        assert np.allclose(v_rot, (x @ w64["v"].T) @ r2d, atol=tol)
        assert np.allclose(v_rot @ f["o"].T, (x @ w64["v"].T @ w64["o"].T) @ r1d, atol=tol)
        h = np.maximum(x @ w64["up"].T, 0.0)
        assert np.allclose(np.maximum(xr @ f["up"].T, 0.0) @ f["down"].T, (h @ w64["down"].T) @ r1d, atol=tol)
