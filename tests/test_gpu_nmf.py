"""Per-tile NMF of |W| by multiplicative updates on the GPU (fp32) against the fp64 CPU oracle, through the C ABI.
Tolerance: the iteration multiplies and divides fp32 sums of up to 1024 terms; after a handful of iterations the
factors are held to 2e-4 relative Frobenius error (measured errors sit near 1e-6)."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _b():
    from paper_1905_05686_b200 import binding
    return binding


SHAPES = [
    # rows, cols, tm, tn, k, iterations
    (2, 2, 2, 2, 1, 1),
    (37, 45, 16, 20, 7, 4),
    (300, 1000, 128, 96, 16, 5),
    (500, 800, 500, 800, 16, 3),
    (512, 1024, 256, 512, 64, 4),
    (384, 776, 384, 776, 145, 2),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_nmf_updates(shape):
    b = _b()
    rows, cols, tm, tn, k, iters = shape
    L = synth.Layer("nmf", rows, cols, tm, tn, k, 0.2, 0.05)
    tiles = L.grid[0] * L.grid[1]
    rng = np.random.default_rng(rows + cols)
    Wb = synth.make_weights(L)
    Mp0 = (rng.random((tiles, tm, k)) * 0.1 + 0.01).astype(np.float32)
    Mz0 = (rng.random((tiles, k, tn)) * 0.1 + 0.01).astype(np.float32)
    want_p, want_z = oracle.nmf_multiplicative(Wb, Mp0, Mz0, tm, tn, iters)
    mp, mz = torch.from_numpy(Mp0.copy()).cuda(), torch.from_numpy(Mz0.copy()).cuda()
    b.lrbi_nmf_update(L, b.to_device_bf16(Wb), mp, mz, iters)
    torch.cuda.synchronize()
    for got, want in ((mp.cpu().numpy().astype(np.float64), want_p), (mz.cpu().numpy().astype(np.float64), want_z)):
        assert np.isfinite(got).all() and (got >= 0).all()
        assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 2e-4
    assert b.device_status() == 0


def test_one_step_by_hand_and_pipeline_into_the_packed_factors():
    b = _b()
    L = synth.Layer("nmf2", 2, 2, 2, 2, 1, 0.5)
    Wb = synth.f32_to_bf16_bits(np.array([[1, -2], [2, 4]], dtype=np.float32))
    mp, mz = torch.ones((1, 2, 1), device="cuda"), torch.ones((1, 1, 2), device="cuda")
    b.lrbi_nmf_update(L, b.to_device_bf16(Wb), mp, mz, 1, eps=0.0)
    assert mz.cpu().numpy().ravel().tolist() == [1.5, 3.0]
    assert np.allclose(mp.cpu().numpy().ravel(), [2 / 3, 4 / 3], rtol=1e-6)
    one = lambda v: torch.tensor([v], dtype=torch.float32, device="cuda")
    ip, iz = b.lrbi_threshold_pack(L, mp, mz, one(1.0), one(2.0))     # Ip = (0, 1)^T, Iz = (0, 1): only |W| = 4 is kept
    mask = b.lrbi_decode_mask(L, ip, iz).cpu().numpy().view(np.uint32)
    assert mask.ravel().tolist() == [0, 2]


def test_nmf_at_the_benchmark_size():
    """Two iterations on the AlexNet layer (144 tiles of 512 x 512, k = 32), the configuration `bench.py` times; this
    is the shape that runs on the cp.async ring kernels."""
    b = _b()
    L = synth.CONFIGS["alexnet_fc"]
    tiles = L.grid[0] * L.grid[1]
    rng = np.random.default_rng(11)
    Wb = synth.make_weights(L)
    Mp0 = (rng.random((tiles, L.tile_rows, L.rank)) * 0.1 + 0.01).astype(np.float32)
    Mz0 = (rng.random((tiles, L.rank, L.tile_cols)) * 0.1 + 0.01).astype(np.float32)
    want_p, want_z = oracle.nmf_multiplicative(Wb, Mp0, Mz0, L.tile_rows, L.tile_cols, 2)
    mp, mz = torch.from_numpy(Mp0.copy()).cuda(), torch.from_numpy(Mz0.copy()).cuda()
    b.lrbi_nmf_update(L, b.to_device_bf16(Wb), mp, mz, 2)
    torch.cuda.synchronize()
    for got, want in ((mp.cpu().numpy().astype(np.float64), want_p), (mz.cpu().numpy().astype(np.float64), want_z)):
        assert np.isfinite(got).all() and (got >= 0).all()
        assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 2e-4
    assert b.device_status() == 0
