"""Generalised layouts: one rank per tile (Section 3.1, last paragraph) and several layers decoded by one launch,
against the CPU oracle, through the C ABI."""
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


def _ranked_case(shape, seed):
    rows, cols, tm, tn, kmax = shape
    L = synth.Layer("ranked", rows, cols, tm, tn, kmax, 0.25, 0.05, (), seed=seed)
    gr, gc = L.grid
    rng = np.random.default_rng(seed)
    Ip, Iz = synth.make_factors(L)
    ranks = rng.integers(1, kmax + 1, gr * gc).astype(np.int32)
    ranks[0] = kmax                                              # the bound itself
    if gr * gc > 2:
        ranks[1] = 0                                             # an empty tile
        ranks[2] = min(kmax, 33)                                 # two words, one bit in the second
    return L, Ip, Iz, ranks


def _dev_ranked(b, Ip, Iz, ranks):
    ipw, izw, ipo, izo = synth.pack_ranked(Ip, Iz, ranks)
    return (torch.from_numpy(ranks).cuda(), torch.from_numpy(ipo).cuda(), torch.from_numpy(izo).cuda(),
            b.to_device_words(ipw), b.to_device_words(izw))


RANKED = [
    # rows, cols, tm, tn, kmax
    (37, 45, 16, 20, 7),
    (300, 1000, 128, 96, 40),
    (512, 1024, 128, 256, 64),
    (640, 1088, 128, 64, 145),
    (1152, 1024, 576, 512, 32),
    (384, 776, 384, 776, 256),
]


@pytest.mark.parametrize("shape", RANKED, ids=lambda s: "x".join(map(str, s)))
def test_ranked_decode_and_product(shape):
    b = _b()
    L, Ip, Iz, ranks = _ranked_case(shape, seed=sum(shape))
    M = oracle.decode_mask_ranks(Ip, Iz, ranks, L.rows, L.cols)
    rk, ipo, izo, ip, iz = _dev_ranked(b, Ip, Iz, ranks)
    got = b.lrbi_decode_mask_ranked(L, rk, ipo, izo, ip, iz).cpu().numpy().view(np.uint32)
    assert (got == synth.pack_mask(M)).all()
    # storage follows the ranks: sum over tiles of ceil(k_t / 32) (tm + tn) words
    want_words = sum(((int(k) + 31) // 32) * (L.tile_rows + L.tile_cols) for k in ranks)
    ipw, izw, _, _ = synth.pack_ranked(Ip, Iz, ranks)
    assert want_words <= ipw.size + izw.size <= want_words + 8
    Wb = synth.make_weights(L)
    W = b.to_device_bf16(Wb)
    for batch in (3, 40, 300):
        Xb = synth.make_activations(L, batch)
        want = oracle.masked_gemm(Wb, M, Xb)
        X = b.to_device_bf16(Xb)
        algos = [b.ALGO_GENERIC, b.ALGO_AUTO]
        if L.cols % 8 == 0 and (L.grid[0] == 1 or L.tile_rows % 128 == 0) and (L.grid[1] == 1 or L.tile_cols % 64 == 0):
            algos += [b.ALGO_TENSOR, b.ALGO_TENSOR_PAIR, b.ALGO_TENSOR_PAIR2, b.ALGO_TENSOR_PAIR192]
        for algo in algos:
            for dt, tol in ((torch.bfloat16, TOL), (torch.float32, TOL_F32)):
                Y = b.lrbi_masked_gemm_ranked(L, rk, ipo, izo, W, ip, iz, X, y_dtype=dt, algo=algo)
                torch.cuda.synchronize()
                got = Y.float().cpu().numpy().astype(np.float64)
                err = np.linalg.norm(got - want) / np.linalg.norm(want)
                assert err <= tol, (b.ALGO_NAMES[algo], batch, str(dt), err)
    assert b.device_status() == 0


def test_equal_ranks_give_the_plain_layout():
    b = _b()
    L = synth.Layer("same", 256, 512, 128, 128, 16, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    ranks = np.full(L.grid[0] * L.grid[1], 16, dtype=np.int32)
    rk, ipo, izo, ip, iz = _dev_ranked(b, Ip, Iz, ranks)
    plain = b.lrbi_decode_mask(L, b.to_device_words(synth.pack_ip(Ip)), b.to_device_words(synth.pack_iz(Iz)))
    assert torch.equal(b.lrbi_decode_mask_ranked(L, rk, ipo, izo, ip, iz), plain)


def test_many_layers_in_one_launch():
    b = _b()
    shapes = [(5, 5, 5, 5, 2), (37, 45, 16, 20, 7), (300, 1000, 128, 96, 16), (256, 512, 128, 64, 33), (64, 4100, 64, 4096, 3)]
    shapes = shapes * 8                                          # 40 layers: two launches (32 + 8)
    layers, ips, izs, wants = [], [], [], []
    for n, (rows, cols, tm, tn, k) in enumerate(shapes):
        L = synth.Layer("batch%d" % n, rows, cols, tm, tn, k, 0.25, 0.05, (), seed=n)
        Ip, Iz = synth.make_factors(L)
        layers.append(L)
        ips.append(b.to_device_words(synth.pack_ip(Ip)))
        izs.append(b.to_device_words(synth.pack_iz(Iz)))
        wants.append(synth.pack_mask(oracle.decode_mask(Ip, Iz, rows, cols)))
    before = b.launch_count()
    masks = b.lrbi_decode_mask_batch(layers, ips, izs)
    assert b.launch_count() - before == 2
    for got, want in zip(masks, wants):
        assert (got.cpu().numpy().view(np.uint32) == want).all()
