"""Decode kernels against the CPU oracle, bit for bit, through the C ABI."""
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


def gpu_decode(layer, Ip, Iz, algo, canary=True):
    b = _b()
    ip = b.to_device_words(synth.pack_ip(Ip))
    iz = b.to_device_words(synth.pack_iz(Iz))
    pitch = (layer.cols + 31) // 32
    n = layer.rows * pitch
    # output sits in the middle of a canary-filled buffer: anything written outside is noticed
    pad = 64
    buf = torch.full((n + 2 * pad,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    out = buf[pad:pad + n].view(layer.rows, pitch)
    b.lrbi_decode_mask(layer, ip, iz, out, algo=algo)
    torch.cuda.synchronize()
    host = buf.cpu().numpy().view(np.uint32)
    assert (host[:pad] == 0x5A5A5A5A).all() and (host[pad + n:] == 0x5A5A5A5A).all(), "wrote outside mask_out"
    return host[pad:pad + n].reshape(layer.rows, pitch)


def check(layer, algo, p=None):
    Ip, Iz = synth.make_factors(layer, p)
    M = oracle.decode_mask(Ip, Iz, layer.rows, layer.cols)
    got = gpu_decode(layer, Ip, Iz, algo)
    want = synth.pack_mask(M)
    xor = got ^ want
    assert synth.popcount_words(xor) == 0, "%d mask bits differ" % synth.popcount_words(xor)
    assert synth.popcount_words(got) == int(M.sum(dtype=np.int64))


ALGOS = ["auto", "ballot", "planes"]


def _algo(name):
    b = _b()
    return {"auto": b.ALGO_AUTO, "ballot": b.ALGO_DECODE_BALLOT, "planes": b.ALGO_DECODE_PLANES,
            "wide": b.ALGO_DECODE_PLANES_WIDE}[name]


@pytest.mark.parametrize("algo", ALGOS)
def test_worked_example_of_the_paper(algo):
    G = read_golden_matrices(os.path.join(GOLDEN, "worked_example.txt"))
    L = synth.Layer("eq5", 5, 5, 5, 5, 2, 0.5)
    if algo == "planes":
        L = synth.Layer("eq5", 5, 5, 5, 32, 2, 0.5)          # planes needs tile_cols % 32 == 0: pad Iz with zero columns
        Iz = np.zeros((1, 1, 2, 32), dtype=np.uint8)
        Iz[0, 0, :, :5] = G["Iz"]
    else:
        Iz = G["Iz"].astype(np.uint8)[None, None]
    Ip = G["Ip"].astype(np.uint8)[None, None]
    got = gpu_decode(L, Ip, Iz, _algo(algo))
    assert (synth.unpack_mask(got, 5) == G["Ia"]).all()
    assert (got >> 5 == 0).all()                               # pad bits are zero


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("name", ["lenet_fc1", "decode_4096"])
def test_paper_configs(name, algo):
    check(synth.CONFIGS[name], _algo(algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_alexnet_and_ffn_index(algo):
    check(synth.CONFIGS["alexnet_fc"], _algo(algo))
    check(synth.Layer("ffn_part", 2048, 4096, 1024, 1024, 64, 0.20), _algo(algo))


RAGGED = [
    # rows, cols, tm, tn, k
    (1, 1, 1, 1, 1),
    (37, 45, 16, 20, 7),          # tn not a multiple of 32: mask words straddle tiles
    (300, 1000, 128, 96, 16),
    (1152, 1024, 576, 512, 32),   # the paper's 576 x 512 AlexNet blocks
    (250, 400, 125, 200, 33),     # 4x4 tiling of FC1, rank not a multiple of 32
    (513, 2100, 512, 1024, 64),
    (260, 300, 130, 150, 145),    # the paper's LSTM rank
    (300, 520, 300, 520, 256),
    (70, 4100, 64, 4096, 3),
    (300, 640, 100, 128, 16),     # 128-column tiles: every 128-column run of a mask row has its own tile
    (1300, 1536, 1300, 768, 40),  # 768-column tiles (runs of two quads), more than 1024 rows per tile
]


@pytest.mark.parametrize("shape", RAGGED, ids=lambda s: "x".join(map(str, s)))
def test_ragged_shapes_ballot(shape):
    rows, cols, tm, tn, k = shape
    check(synth.Layer("rag", rows, cols, tm, tn, k, 0.2), _algo("ballot"))


@pytest.mark.parametrize("shape", [s for s in RAGGED if s[3] % 32 == 0] + [(1000, 2080, 250, 416, 16), (2100, 96, 2100, 32, 9)],
                         ids=lambda s: "x".join(map(str, s)))
def test_ragged_shapes_planes(shape):
    rows, cols, tm, tn, k = shape
    check(synth.Layer("rag", rows, cols, tm, tn, k, 0.2), _algo("planes"))


def _wide_covers(s):
    """tiles of 128, 256 or 512 columns, of a multiple of 1024 columns, or one tile column of a multiple of 128; rank <= 256"""
    rows, cols, tm, tn, k = s
    return k <= 256 and tn % 128 == 0 and (cols <= tn or tn % 1024 == 0 or tn in (128, 256, 512))


def test_wide_variant_refuses_other_tile_widths():
    b = _b()
    L = synth.Layer("rag", 1300, 1536, 1300, 768, 40, 0.2)      # two tile columns of 768
    Ip, Iz = synth.make_factors(L)
    with pytest.raises(b.LrbiError) as e:
        gpu_decode(L, Ip, Iz, b.ALGO_DECODE_PLANES_WIDE)
    assert e.value.code == b.ERR_UNSUPPORTED
    check(L, b.ALGO_AUTO)                                        # the automatic choice still covers it


@pytest.mark.parametrize("shape", [s for s in RAGGED if _wide_covers(s)] +
                         [(1300, 768, 1300, 768, 40), (700, 5120, 350, 512, 8), (300, 2304, 100, 256, 3), (5000, 8192, 2500, 1024, 5),
                          (4096, 4096, 256, 256, 8), (2100, 3072, 1050, 1024, 64), (600, 2304, 128, 256, 16)],
                         ids=lambda s: "x".join(map(str, s)))
def test_ragged_shapes_planes_wide(shape):
    rows, cols, tm, tn, k = shape
    check(synth.Layer("rag", rows, cols, tm, tn, k, 0.2), _algo("wide"))


def test_planes_refuses_unaligned_tiles():
    b = _b()
    L = synth.Layer("rag", 37, 45, 16, 20, 7, 0.2)
    Ip, Iz = synth.make_factors(L)
    with pytest.raises(b.LrbiError) as e:
        gpu_decode(L, Ip, Iz, b.ALGO_DECODE_PLANES)
    assert e.value.code == b.ERR_UNSUPPORTED


@pytest.mark.parametrize("algo", ["ballot", "planes", "wide"])
def test_degenerate_factors(algo):
    L = synth.Layer("deg", 96, 160, 32, 32, 5, 0.2) if algo != "wide" else synth.Layer("deg", 96, 640, 32, 128, 5, 0.2)
    for p in (0.0, 1.0):
        check(L, _algo(algo), p=p)                              # empty and full masks


@pytest.mark.parametrize("algo", ["ballot", "planes", "wide"])
def test_bits_beyond_rank_are_ignored(algo):
    b = _b()
    L = synth.Layer("pad", 64, 96, 32, 32, 5, 0.3) if algo != "wide" else synth.Layer("pad", 64, 384, 32, 128, 5, 0.3)
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    ipw = synth.pack_ip(Ip) | np.uint32(0xFFFFFFE0)            # garbage in bits >= k of both factors
    izw = synth.pack_iz(Iz) | np.uint32(0xFFFFFFE0)
    out = b.lrbi_decode_mask(L, b.to_device_words(ipw), b.to_device_words(izw), algo=_algo(algo))
    got = out.cpu().numpy().view(np.uint32)
    assert (got == synth.pack_mask(M)).all()
