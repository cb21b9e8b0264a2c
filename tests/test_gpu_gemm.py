"""Fused decode + masked GEMM kernels against the fp64 CPU oracle, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

# Tolerance of the comparison with the fp64 oracle: relative Frobenius error.  fp32 accumulation of
# K <= 9216 products contributes ~1e-6; rounding Y to bf16 contributes about 2^-9 / sqrt(3) = 1.1e-3
# (uniform rounding error of half an ulp, relative); 5e-3 leaves a factor of four above that.
TOL = 5e-3
TOL_F32 = 2e-5


def _b():
    from paper_1905_05686_b200 import binding
    return binding


def rel_fro(got, want):
    n = np.linalg.norm(want)
    if n == 0:
        return 0.0 if not np.any(got) else np.inf
    return float(np.linalg.norm(got - want) / n)


class Case:
    def __init__(self, layer, batch, p=None):
        b = _b()
        self.layer, self.batch = layer, batch
        self.Ip, self.Iz = synth.make_factors(layer, p)
        self.Wb = synth.make_weights(layer)
        self.Xb = synth.make_activations(layer, batch)
        self.ip = b.to_device_words(synth.pack_ip(self.Ip))
        self.iz = b.to_device_words(synth.pack_iz(self.Iz))
        self.W = b.to_device_bf16(self.Wb)
        self.X = b.to_device_bf16(self.Xb)

    def run(self, algo, y_dtype=None):
        b = _b()
        y_dtype = y_dtype or torch.bfloat16
        pad = 256
        n = self.batch * self.layer.rows
        canary = 1.0e30 if y_dtype == torch.float32 else 1.0e30
        buf = torch.full((n + 2 * pad,), canary, dtype=y_dtype, device="cuda")
        Y = buf[pad:pad + n].view(self.batch, self.layer.rows)
        b.lrbi_masked_gemm(self.layer, self.W, self.ip, self.iz, self.X, Y=Y, algo=algo)
        torch.cuda.synchronize()
        assert b.device_status() == 0
        host = buf.float().cpu().numpy()
        assert (host[:pad] > 1e29).all() and (host[pad + n:] > 1e29).all(), "wrote outside Y"
        return host[pad:pad + n].reshape(self.batch, self.layer.rows).astype(np.float64)

    def oracle_full(self):
        M = oracle.decode_mask(self.Ip, self.Iz, self.layer.rows, self.layer.cols)
        return oracle.masked_gemm(self.Wb, M, self.Xb)

    def oracle_samples(self, n, seed=0):
        rng = np.random.default_rng(seed)
        b_idx = rng.integers(0, self.batch, n)
        o_idx = rng.integers(0, self.layer.rows, n)
        # always include the corners and the last row/column of every 128-block boundary
        b_idx[:4] = [0, 0, self.batch - 1, self.batch - 1]
        o_idx[:4] = [0, self.layer.rows - 1, 0, self.layer.rows - 1]
        return b_idx, o_idx, oracle.masked_gemm_samples(self.Wb, self.Ip, self.Iz, self.Xb, b_idx, o_idx)


def algos_for(layer, batch):
    b = _b()
    out = [b.ALGO_GENERIC, b.ALGO_AUTO]
    from paper_1905_05686_b200.binding import ALGO_GEMV, ALGO_TENSOR
    if batch <= 8 and layer.cols % 8 == 0 and layer.tile_cols % 8 == 0 and layer.kw <= 2:
        out.append(ALGO_GEMV)
    return out


SMALL = [
    # rows, cols, tm, tn, k, batch
    (5, 5, 5, 5, 2, 3),
    (37, 45, 16, 20, 7, 5),
    (300, 1000, 128, 96, 16, 4),
    (250, 400, 125, 200, 33, 9),
    (260, 304, 130, 152, 145, 2),
    (256, 512, 128, 64, 16, 1),
    (256, 512, 128, 64, 16, 8),
    (384, 1024, 128, 256, 64, 3),
    (500, 800, 500, 800, 16, 2),
]


@pytest.mark.parametrize("shape", SMALL, ids=lambda s: "x".join(map(str, s)))
def test_small_shapes_every_kernel_that_covers_them(shape):
    b = _b()
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("small", rows, cols, tm, tn, k, 0.25, 0.05)
    c = Case(L, batch)
    want = c.oracle_full()
    tried = 0
    for algo in (b.ALGO_GENERIC, b.ALGO_GEMV, b.ALGO_STREAM, b.ALGO_TENSOR, b.ALGO_AUTO):
        try:
            got = c.run(algo)
        except b.LrbiError as e:
            assert e.code == b.ERR_UNSUPPORTED and algo in (b.ALGO_GEMV, b.ALGO_STREAM, b.ALGO_TENSOR)
            continue
        tried += 1
        assert rel_fro(got, want) <= TOL, (b.ALGO_NAMES[algo], rel_fro(got, want))
        got32 = c.run(algo, torch.float32)
        assert rel_fro(got32, want) <= TOL_F32, (b.ALGO_NAMES[algo], rel_fro(got32, want))
    assert tried >= 2


TC_SHAPES = [
    # rows, cols, tm, tn, k, batch  -- several 128-row blocks, ragged tails in every dimension
    (128, 64, 128, 64, 8, 16),
    (256, 512, 128, 64, 16, 24),
    (500, 800, 500, 800, 16, 32),
    (640, 1088, 128, 64, 33, 100),
    (384, 2048, 128, 512, 64, 129),
    (256, 2304, 128, 256, 16, 700),
    (1152, 1024, 128, 512, 32, 300),
    (1024, 4096, 512, 1024, 64, 520),
    (256, 1024, 128, 256, 145, 64),      # the paper's LSTM rank: five index words per row
    (384, 776, 384, 776, 256, 40),       # one tile, rank 256, ragged last K block
    (256, 640, 128, 128, 16, 260),       # 128-column tiles: 64-column panels
]


@pytest.mark.parametrize("shape", TC_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_tensor_core_kernel(shape):
    b = _b()
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("tc", rows, cols, tm, tn, k, 0.25, 0.05)
    c = Case(L, batch)
    want = c.oracle_full()
    got = c.run(b.ALGO_TENSOR)
    assert rel_fro(got, want) <= TOL, rel_fro(got, want)
    got32 = c.run(b.ALGO_TENSOR, torch.float32)
    assert rel_fro(got32, want) <= TOL_F32, rel_fro(got32, want)


STREAM_SHAPES = [
    # rows, cols, tm, tn, k, batch
    (16, 32, 16, 32, 4, 1),
    (500, 800, 500, 800, 16, 7),          # ragged rows, 800 = 25 steps of 32
    (500, 808, 500, 808, 16, 9),          # last step has columns in one lane group only
    (384, 1024, 128, 256, 64, 16),
    (640, 1088, 128, 64, 33, 17),
    (1024, 4096, 512, 1024, 64, 32),
    (272, 2304, 16, 256, 16, 5),
]


@pytest.mark.parametrize("shape", STREAM_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_stream_kernel(shape):
    b = _b()
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("stream", rows, cols, tm, tn, k, 0.25, 0.05)
    c = Case(L, batch)
    want = c.oracle_full()
    got = c.run(b.ALGO_STREAM)
    assert rel_fro(got, want) <= TOL, rel_fro(got, want)
    got32 = c.run(b.ALGO_STREAM, torch.float32)
    assert rel_fro(got32, want) <= TOL_F32, rel_fro(got32, want)


def test_mask_alignment_with_one_hot_activations():
    """A one-hot X row returns a masked column of W exactly (bf16 values pass through unrounded)."""
    b = _b()
    L = synth.Layer("onehot", 384, 1024, 128, 256, 16, 0.3, 0.05)
    c = Case(L, 40)
    cols_hit = np.arange(40) * 25 + 3
    X = np.zeros((40, L.cols), dtype=np.float32)
    X[np.arange(40), cols_hit] = 1.0
    c.Xb = synth.f32_to_bf16_bits(X)
    c.X = b.to_device_bf16(c.Xb)
    M = oracle.decode_mask(c.Ip, c.Iz, L.rows, L.cols)
    want = (synth.bf16_bits_to_f32(c.Wb) * M)[:, cols_hit].T.astype(np.float64)
    for algo in (b.ALGO_GENERIC, b.ALGO_TENSOR):
        assert (c.run(algo) == want).all()
    c2 = Case(L, 8)
    c2.Xb = c.Xb[:8].copy()
    c2.X = b.to_device_bf16(c2.Xb)
    assert (c2.run(b.ALGO_GEMV) == want[:8]).all()


def test_degenerate_masks_and_poisoned_pruned_weights():
    b = _b()
    L = synth.Layer("deg", 256, 512, 128, 128, 16, 0.2, 0.05)
    for batch, algo in ((4, b.ALGO_GEMV), (48, b.ALGO_TENSOR), (3, b.ALGO_GENERIC)):
        c = Case(L, batch, p=0.0)                               # nothing kept: Y is exactly zero
        assert not c.run(algo).any()
        c = Case(L, batch, p=1.0)                               # everything kept: plain X W^T
        W = synth.bf16_bits_to_f32(c.Wb).astype(np.float64)
        X = synth.bf16_bits_to_f32(c.Xb).astype(np.float64)
        assert rel_fro(c.run(algo), X @ W.T) <= TOL
        c = Case(L, batch)                                      # NaN / Inf parked in pruned weights never reach Y
        M = oracle.decode_mask(c.Ip, c.Iz, L.rows, L.cols)
        want = c.oracle_full()
        Wb = c.Wb.copy()
        Wb[M == 0] = np.where(np.arange((M == 0).sum()) % 2 == 0, 0x7FC0, 0x7F80).astype(np.uint16)
        c.Wb, c.W = Wb, b.to_device_bf16(Wb)
        got = c.run(algo)
        assert np.isfinite(got).all() and rel_fro(got, want) <= TOL


def test_lenet_fc1_config():
    b = _b()
    L = synth.CONFIGS["lenet_fc1"]
    c = Case(L, 32)
    want = c.oracle_full()
    for algo in (b.ALGO_AUTO, b.ALGO_TENSOR, b.ALGO_GENERIC):
        assert rel_fro(c.run(algo), want) <= TOL


@pytest.mark.parametrize("batch", [1, 16, 128])
def test_alexnet_fc_config(batch):
    b = _b()
    L = synth.CONFIGS["alexnet_fc"]
    c = Case(L, batch)
    got = c.run(b.ALGO_AUTO)
    if batch <= 16:
        want = c.oracle_full()
        assert rel_fro(got, want) <= TOL
    else:
        M = oracle.decode_mask(c.Ip, c.Iz, L.rows, L.cols)
        rows_b = [0, 1, 63, 64, 127]
        want = oracle.masked_gemm(c.Wb, M, c.Xb[rows_b])
        assert rel_fro(got[rows_b], want) <= TOL
    b_idx, o_idx, ys = c.oracle_samples(2000, seed=batch)
    assert rel_fro(got[b_idx, o_idx], ys) <= TOL


def test_conv3x3_config():
    b = _b()
    L = synth.CONFIGS["conv3x3_256"]
    c = Case(L, 12544)
    got = c.run(b.ALGO_AUTO)
    M = oracle.decode_mask(c.Ip, c.Iz, L.rows, L.cols)
    rows_b = [0, 127, 128, 255, 256, 6271, 12543 - 255, 12543]
    want = oracle.masked_gemm(c.Wb, M, c.Xb[rows_b])
    assert rel_fro(got[rows_b], want) <= TOL
    b_idx, o_idx, ys = c.oracle_samples(20000)
    assert rel_fro(got[b_idx, o_idx], ys) <= TOL
    # property that holds at any size: a column of Y whose mask row is empty is exactly zero
    empty_rows = np.flatnonzero(M.sum(axis=1) == 0)
    assert not got[:, empty_rows].any()


def test_ffn_config_sampled():
    b = _b()
    L = synth.CONFIGS["ffn_16384x4096"]
    c = Case(L, 4096)
    got = c.run(b.ALGO_AUTO)
    b_idx, o_idx, ys = c.oracle_samples(40000)
    assert rel_fro(got[b_idx, o_idx], ys) <= TOL
    # two full batch rows and two full output columns
    M = oracle.decode_mask(c.Ip, c.Iz, L.rows, L.cols)
    want = oracle.masked_gemm(c.Wb, M, c.Xb[[0, 4095]])
    assert rel_fro(got[[0, 4095]], want) <= TOL
    # linearity in X: doubling the activations doubles Y exactly (power of two scaling is exact in bf16/fp32)
    c.Xb = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(c.Xb) * np.float32(2.0))
    c.X = b.to_device_bf16(c.Xb)
    got2 = c.run(b.ALGO_AUTO)
    assert (got2[:64] == 2.0 * got[:64]).all()
