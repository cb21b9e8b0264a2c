"""Inner loop of Algorithm 1 on the GPU (binary conversion into packed factors, per-tile index counts and
cost) against the CPU oracle, through the C ABI.  Bits and counts must agree exactly; the cost is a sum of
bf16 magnitudes accumulated in fp32 over up to 32 weights and in fp64 beyond, held to 1e-6 relative."""
import os

import numpy as np
import pytest

import oracle
from conftest import GOLDEN, read_golden_matrices
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _b():
    from paper_1905_05686_b200 import binding
    return binding


def _factors(rng, tiles, tm, tn, k):
    Mp = rng.random((tiles, tm, k), dtype=np.float32) * rng.random((tiles, 1, 1), dtype=np.float32) * 2
    Mz = rng.random((tiles, k, tn), dtype=np.float32)
    # exact ties with the thresholds below must go the ">=" way on both sides
    Mp[:, ::3, ::2] = 0.5
    Mz[:, ::2, ::5] = 0.25
    return Mp, Mz


SHAPES = [
    # rows, cols, tm, tn, k
    (5, 5, 5, 5, 2),
    (37, 45, 16, 20, 7),
    (300, 1000, 128, 96, 16),
    (250, 400, 125, 200, 33),
    (260, 304, 130, 152, 145),
    (512, 1024, 256, 256, 8),
    (1152, 1024, 576, 512, 32),
    (384, 776, 384, 776, 256),
    (1024, 2048, 1024, 1024, 64),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_threshold_pack_and_index_cost(shape):
    b = _b()
    rows, cols, tm, tn, k = shape
    L = synth.Layer("alg1", rows, cols, tm, tn, k, 0.2, 0.05)
    gr, gc = L.grid
    tiles = gr * gc
    rng = np.random.default_rng(rows * 31 + cols)
    Mp, Mz = _factors(rng, tiles, tm, tn, k)
    Tp = (0.3 + 0.4 * rng.random(tiles)).astype(np.float32)
    Tz = (0.15 + 0.2 * rng.random(tiles)).astype(np.float32)
    Tp[0], Tz[0] = 0.5, 0.25                                     # the tie values
    if tiles > 2:
        Tp[1] = np.inf                                           # an empty Ip: nothing of that tile is kept
    # --- binary conversion
    Ip = oracle.threshold(Mp, Tp).reshape(gr, gc, tm, k)
    Iz = oracle.threshold(Mz, Tz).reshape(gr, gc, k, tn)
    ip, iz = b.lrbi_threshold_pack(L, torch.from_numpy(Mp).cuda(), torch.from_numpy(Mz).cuda(),
                                   torch.from_numpy(Tp).cuda(), torch.from_numpy(Tz).cuda())
    assert (ip.cpu().numpy().view(np.uint32) == synth.pack_ip(Ip)).all()
    assert (iz.cpu().numpy().view(np.uint32) == synth.pack_iz(Iz)).all()
    # --- counts and cost of that candidate
    Wb = synth.make_weights(L)
    Wb[0, 0] = 0x7FC0                                            # a NaN weight counts as pruned
    theta = float(np.float32(0.06))
    Ia = oracle.decode_mask(Ip, Iz, rows, cols)
    kept_i, kept_a, lost, cost = oracle.index_cost(Wb, theta, Ia, tm, tn)
    out = b.lrbi_index_cost(L, b.to_device_bf16(Wb), theta, ip, iz)
    torch.cuda.synchronize()
    g_i, g_a, g_l, g_c = b.tile_costs(out)
    assert (g_i == kept_i).all() and (g_a == kept_a).all() and (g_l == lost).all()
    assert np.allclose(g_c, cost, rtol=1e-6, atol=0)
    assert (g_c[lost == 0] == 0).all()
    # a second call overwrites the records (they start from zero again)
    out2 = b.lrbi_index_cost(L, b.to_device_bf16(Wb), theta, ip, iz, out=out)
    assert (b.tile_costs(out2)[2] == lost).all()
    assert b.device_status() == 0


def test_papers_example_through_the_gpu():
    b = _b()
    G = read_golden_matrices(os.path.join(GOLDEN, "worked_example.txt"))
    L = synth.Layer("eq4", 5, 5, 5, 5, 2, 0.5)
    one = lambda v: torch.tensor([v], dtype=torch.float32, device="cuda")
    ip, iz = b.lrbi_threshold_pack(L, torch.from_numpy(G["Mp"].astype(np.float32)[None]).cuda(),
                                   torch.from_numpy(G["Mz"].astype(np.float32)[None]).cuda(), one(0.5), one(0.6))
    assert (ip.cpu().numpy().view(np.uint32) == synth.pack_ip(G["Ip"].astype(np.uint8)[None, None])).all()   # Eq. 5
    assert (iz.cpu().numpy().view(np.uint32) == synth.pack_iz(G["Iz"].astype(np.uint8)[None, None])).all()
    Wb = synth.f32_to_bf16_bits(G["W"].astype(np.float32))
    theta = float(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.array([0.7], dtype=np.float32)))[0])
    # 5 columns: not a multiple of 8, the any-shape path
    g_i, g_a, g_l, g_c = b.tile_costs(b.lrbi_index_cost(L, b.to_device_bf16(Wb), theta, ip, iz))
    assert (g_i[0], g_a[0], g_l[0], g_c[0]) == (13, 15, 0, 0.0)   # S = 12/25, S_a = 10/25, nothing lost


def test_search_driven_by_the_gpu_kernels_matches_the_oracle_search():
    """Algorithm 1's sweep with every conversion, decode, count and cost taken from the GPU: the same candidates,
    the same costs and the same choice as the oracle's search on the same factors."""
    b = _b()
    rng = np.random.default_rng(3)
    m, n, k = 64, 96, 8
    L = synth.Layer("search", m, n, m, n, k, 0.2, 0.05)
    Wb = synth.f32_to_bf16_bits((rng.standard_normal((m, n)) * 0.05).astype(np.float32))
    A = np.abs(synth.bf16_bits_to_f32(Wb))
    # factors that carry some of |W|'s structure: a few multiplicative updates from a random start
    Mp, Mz = rng.random((m, k)).astype(np.float32) + 0.1, rng.random((k, n)).astype(np.float32) + 0.1
    for _ in range(30):
        Mz *= (Mp.T @ A) / (Mp.T @ Mp @ Mz + 1e-9)
        Mp *= (A @ Mz.T) / (Mp @ Mz @ Mz.T + 1e-9)
    theta = float(np.float32(np.quantile(A, 0.8)))
    ref = oracle.alg1_search(Wb, theta, Mp, Mz, sp_step=0.1, tol=2e-3, max_iter=16)

    W = b.to_device_bf16(Wb)
    mp, mz = torch.from_numpy(Mp[None].copy()).cuda(), torch.from_numpy(Mz[None].copy()).cuda()
    dev = lambda v: torch.tensor([v], dtype=torch.float32, device="cuda")
    full = b.lrbi_threshold_pack(L, mp, mz, dev(-1.0), dev(-1.0))
    S = 1.0 - b.tile_costs(b.lrbi_index_cost(L, W, theta, *full))[0][0] / float(m * n)
    assert S == ref["S"]
    best, tried = None, []
    for step in range(11):
        Sp = min(step * 0.1, 1.0)
        Sz = 0.0 if Sp >= 1.0 else min(max(oracle.sz_from_eq7(S, Sp, k), 0.0), 1.0)
        Tp = oracle.threshold_for_sparsity(Mp, Sp)             # host logic of the search: order statistics of the factors
        lo, hi = 0.0, 1.0
        for _ in range(16):
            Tz = oracle.threshold_for_sparsity(Mz, Sz)
            ip, iz = b.lrbi_threshold_pack(L, mp, mz, dev(float(Tp)), dev(float(Tz)))
            _, kept_a, lost, cost = b.tile_costs(b.lrbi_index_cost(L, W, theta, ip, iz))
            Sa = 1.0 - kept_a[0] / float(m * n)
            if abs(Sa - S) <= 2e-3:
                break
            if Sa > S:
                hi = Sz
            else:
                lo = Sz
            Sz = 0.5 * (lo + hi)
        tried.append((Sp, Sz, float(cost[0]), Sa, int(lost[0])))
        if best is None or best[2] > cost[0]:
            best = tried[-1]
    for got, want in zip(tried, ref["tried"]):
        assert got[0] == pytest.approx(want["Sp"]) and got[1] == want["Sz"] and got[4] == want["lost"]
        assert got[2] == pytest.approx(want["cost"], rel=1e-6) and got[3] == want["Sa"]
    assert best[0] == pytest.approx(ref["best"]["Sp"]) and best[1] == ref["best"]["Sz"]


@pytest.mark.parametrize("name", ["alexnet_fc", "ffn_16384x4096"])
def test_index_cost_at_the_benchmark_sizes(name):
    """The two layers `bench.py` times the cost evaluation on, whole: every tile's counts exactly, its cost to 1e-6."""
    b = _b()
    L = synth.CONFIGS[name]
    Ip, Iz = synth.make_factors(L)
    Wb = synth.make_weights(L)
    theta = float(np.float32(1.3 * L.w_std))
    Ia = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    kept_i, kept_a, lost, cost = oracle.index_cost(Wb, theta, Ia, L.tile_rows, L.tile_cols)
    out = b.lrbi_index_cost(L, b.to_device_bf16(Wb), theta, b.to_device_words(synth.pack_ip(Ip)), b.to_device_words(synth.pack_iz(Iz)))
    torch.cuda.synchronize()
    g_i, g_a, g_l, g_c = b.tile_costs(out)
    assert kept_i.sum() > 0 and lost.sum() > 0                   # the threshold cuts inside the distribution
    assert (g_i == kept_i).all() and (g_a == kept_a).all() and (g_l == lost).all()
    assert np.allclose(g_c, cost, rtol=1e-6, atol=0)
    assert b.device_status() == 0
