"""Backward pass of the masked layer (dX, dW) against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

TOL, TOL_F32 = 5e-3, 2e-5


def _b():
    from paper_1905_05686_b200 import binding
    return binding


def rel_fro(got, want):
    n = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / n) if n else (0.0 if not np.any(got) else np.inf)


def test_transpose_is_exact():
    b = _b()
    rng = np.random.default_rng(1)
    for rows, cols in [(1, 1), (5, 70), (64, 64), (130, 257), (1000, 24), (72, 136), (512, 1032), (8, 8)]:
        a = rng.integers(0, 2**16, (rows, cols), dtype=np.uint16)
        got = b.lrbi_transpose_bf16(b.to_device_bf16(a)).view(torch.int16).cpu().numpy().view(np.uint16)
        assert (got == a.T).all()


SHAPES = [
    # rows, cols, tm, tn, k, batch
    (37, 45, 16, 20, 7, 5),               # nothing aligned: the any-shape kernels
    (300, 1000, 128, 96, 16, 9),
    (256, 512, 128, 128, 16, 64),         # tensor-core shapes in both directions
    (640, 1024, 128, 256, 33, 264),
    (1024, 768, 512, 128, 64, 520),
    (384, 776, 384, 776, 256, 40),        # one tile
    (512, 2048, 256, 1024, 145, 136),
    (1000, 1304, 1000, 1304, 20, 72),     # one tile, nothing a multiple of 64: ragged 64 x 64 boxes of the MN-major dW on every side
    (2048, 520, 512, 520, 9, 1032),       # dW tiles of 256 x 512 outputs with a ragged third row pair; K = 16 blocks + 8
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_masked_backward(shape):
    b = _b()
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("bwd", rows, cols, tm, tn, k, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, rows, cols)
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, batch)
    dYb = synth.make_activations(synth.Layer("bwd_dy", cols, rows, tn, tm, k, 0.25, 0.05), batch)   # [batch, rows]
    want_dX, want_dW = oracle.masked_backward(Wb, M, Xb, dYb)
    ip, iz = b.to_device_words(synth.pack_ip(Ip)), b.to_device_words(synth.pack_iz(Iz))
    W, X, dY = b.to_device_bf16(Wb), b.to_device_bf16(Xb), b.to_device_bf16(dYb)
    Wt = b.lrbi_transpose_bf16(W)
    tc_ok = rows % 8 == 0 and (L.grid[1] == 1 or tn % 128 == 0) and (L.grid[0] == 1 or tm % 64 == 0)
    algos = [b.ALGO_GENERIC, b.ALGO_AUTO] + ([b.ALGO_TENSOR, b.ALGO_TENSOR_PAIR, b.ALGO_TENSOR_PAIR2, b.ALGO_TENSOR_PAIR192] if tc_ok else [])
    for algo in algos:
        for dt, tol in ((torch.bfloat16, TOL), (torch.float32, TOL_F32)):
            got = b.lrbi_masked_gemm_dx(L, Wt, ip, iz, dY, dtype=dt, algo=algo).float().cpu().numpy().astype(np.float64)
            assert rel_fro(got, want_dX) <= tol, ("dX", b.ALGO_NAMES[algo], str(dt), rel_fro(got, want_dX))
    if tc_ok:                                                    # the automatic choice took the tensor-core kernel
        before = b.launch_count()
        b.lrbi_masked_gemm_dx(L, Wt, ip, iz, dY)
        assert b.launch_count() - before <= 2
    for ws in ("auto", None):
        for dt, tol in ((torch.bfloat16, TOL), (torch.float32, TOL_F32)):
            got = b.lrbi_masked_gemm_dw(L, dY, X, ip, iz, dtype=dt, workspace=ws).float().cpu().numpy().astype(np.float64)
            assert rel_fro(got, want_dW) <= tol, ("dW", ws, str(dt), rel_fro(got, want_dW))
            assert not got[M == 0].any()                         # a pruned weight gets no gradient, exactly
    # aligned layers: one launch, the persistent pair kernel on X and dY as they are (MN-major operands), no copies
    gr, gc = L.grid
    if rows % 8 == 0 and cols % 8 == 0 and batch % 8 == 0 and (gc == 1 or tn % 128 == 0) and (gr == 1 or tm % 256 == 0):
        before = b.launch_count()
        b.lrbi_masked_gemm_dw(L, dY, X, ip, iz, workspace=None)
        assert b.launch_count() - before == 1
    assert b.device_status() == 0


def test_poisoned_pruned_weights_do_not_reach_dx():
    b = _b()
    L = synth.Layer("bwd_nan", 256, 512, 128, 128, 16, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, 200)
    dYb = synth.make_activations(synth.Layer("bwd_dy", L.cols, L.rows, 128, 128, 16, 0.25, 0.05), 200)
    want, _ = oracle.masked_backward(Wb, M, Xb, dYb)
    Wb2 = Wb.copy()
    Wb2[M == 0] = 0x7FC0
    ip, iz = b.to_device_words(synth.pack_ip(Ip)), b.to_device_words(synth.pack_iz(Iz))
    Wt = b.lrbi_transpose_bf16(b.to_device_bf16(Wb2))
    got = b.lrbi_masked_gemm_dx(L, Wt, ip, iz, b.to_device_bf16(dYb)).float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all() and rel_fro(got, want) <= TOL


def test_backward_at_the_benchmark_size_on_sampled_rows():
    """dX and dW of the FFN layer at batch 4096, the calls `bench.py` times (dX on the persistent pair kernel, dW on
    the same kernel with MN-major operands, one launch).  A row of dX depends on one row of dY and a row of dW on one
    column of dY, so the oracle computes a sample of rows of each from the matching slices of the inputs."""
    b = _b()
    L = synth.CONFIGS["ffn_16384x4096"]
    batch = 4096
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, batch)
    dYb = synth.make_activations(synth.Layer("bwd_dy", L.cols, L.rows, L.tile_cols, L.tile_rows, L.rank, 0.2, 0.02), batch)   # [batch, rows]
    ip, iz = b.to_device_words(synth.pack_ip(Ip)), b.to_device_words(synth.pack_iz(Iz))
    W, X, dY = b.to_device_bf16(Wb), b.to_device_bf16(Xb), b.to_device_bf16(dYb)
    rng = np.random.default_rng(7)
    # --- dX: sampled batch rows (first and last included)
    bs = np.unique(np.concatenate([[0, batch - 1], rng.integers(0, batch, 22)]))
    want_dX, _ = oracle.masked_backward(Wb, M, Xb[bs], dYb[bs])
    Wt = b.lrbi_transpose_bf16(W)
    before = b.launch_count()
    got = b.lrbi_masked_gemm_dx(L, Wt, ip, iz, dY, dtype=torch.float32)
    assert b.launch_count() - before == 1
    assert rel_fro(got[torch.from_numpy(bs).cuda()].cpu().numpy().astype(np.float64), want_dX) <= TOL_F32
    del got, Wt
    # --- dW: sampled rows of the layer, from every tile row and both CTAs of a pair
    os_ = np.unique(np.concatenate([[0, 127, 128, 255, 256, L.rows - 1], rng.integers(0, L.rows, 26)]))
    _, want_dW = oracle.masked_backward(Wb[os_], M[os_], Xb, np.ascontiguousarray(dYb[:, os_]))
    before = b.launch_count()
    got = b.lrbi_masked_gemm_dw(L, dY, X, ip, iz, dtype=torch.float32, workspace=None)
    assert b.launch_count() - before == 1
    got = got[torch.from_numpy(os_).cuda()].cpu().numpy().astype(np.float64)
    assert rel_fro(got, want_dW) <= TOL_F32
    assert not got[M[os_] == 0].any()
    assert b.device_status() == 0
