"""Seeded random layouts (ragged tiles, odd ranks, odd batches) through every kernel that accepts them,
against the CPU oracle.  Small sizes: the point is the corner cases of the index arithmetic."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
TOL = 5e-3


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        tm = int(rng.choice([16, 32, 48, 100, 128, 130, 256]))
        tn = int(rng.choice([8, 32, 40, 64, 96, 128, 256, 320]))
        gr, gc = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        rows = tm * gr - int(rng.integers(0, min(tm, 20))) if rng.random() < 0.5 else tm * gr
        cols = tn * gc - 8 * int(rng.integers(0, max(1, min(tn // 8, 4)))) if rng.random() < 0.5 else tn * gc
        k = int(rng.choice([1, 3, 8, 16, 31, 32, 33, 64, 65, 100]))
        batch = int(rng.choice([1, 2, 3, 5, 8, 9, 17, 40, 129, 300]))
        out.append((max(rows, 1), max(cols, 8), tm, tn, k, batch))
    return out


@pytest.mark.parametrize("shape", _cases(24, 2024), ids=lambda s: "x".join(map(str, s)))
def test_random_layouts(shape):
    from paper_1905_05686_b200 import binding as B
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("fuzz", rows, cols, tm, tn, k, 0.3, 0.05, (), seed=rows * 7 + cols)
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, rows, cols)
    ip, iz = B.to_device_words(synth.pack_ip(Ip)), B.to_device_words(synth.pack_iz(Iz))
    want_mask = synth.pack_mask(M)
    ran = 0
    for algo in (B.ALGO_DECODE_BALLOT, B.ALGO_DECODE_PLANES, B.ALGO_DECODE_PLANES_WIDE, B.ALGO_AUTO):
        try:
            got = B.lrbi_decode_mask(L, ip, iz, algo=algo).cpu().numpy().view(np.uint32)
        except B.LrbiError as e:
            assert e.code == B.ERR_UNSUPPORTED and algo != B.ALGO_DECODE_BALLOT
            continue
        ran += 1
        assert (got == want_mask).all(), B.ALGO_NAMES[algo]
    assert ran >= 2
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, batch)
    W, X = B.to_device_bf16(Wb), B.to_device_bf16(Xb)
    want = oracle.masked_gemm(Wb, M, Xb)
    ran = 0
    for algo in (B.ALGO_GENERIC, B.ALGO_GEMV, B.ALGO_STREAM, B.ALGO_TENSOR, B.ALGO_AUTO):
        try:
            Y = B.lrbi_masked_gemm(L, W, ip, iz, X, algo=algo)
        except B.LrbiError as e:
            assert e.code == B.ERR_UNSUPPORTED and algo not in (B.ALGO_GENERIC, B.ALGO_AUTO)
            continue
        ran += 1
        got = Y.float().cpu().numpy().astype(np.float64)
        nrm = np.linalg.norm(want)
        if nrm == 0:
            assert not got.any()
        else:
            assert np.linalg.norm(got - want) / nrm <= TOL, B.ALGO_NAMES[algo]
    assert ran >= 2
    assert B.device_status() == 0
