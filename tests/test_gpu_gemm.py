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


def assert_elementwise(got, want, Xb, Wb, M, bf16_out, what=""):
    """Every output element, not only the norm of the difference.

    bf16 output is one rounding of the fp32 sum: half an ulp, 2^-9 relative; 2^-8 is allowed.  The fp32
    sum itself differs from the fp64 one by accumulation error, which scales with sum_i |x_i w_i| over
    the kept weights; that sum is bounded by A = ||x_b|| * ||(w .* m)_o|| (Cauchy-Schwarz), and 2^-14 A is
    allowed (measured fp32-output errors sit two orders of magnitude below it).  A single wrong, missing
    or extra product moves an element by about A / sqrt(K * density * K), far outside this bound, and so does
    a 16-byte chunk written to the wrong place.
    """
    xn = np.linalg.norm(synth.bf16_bits_to_f32(Xb).astype(np.float64), axis=1)
    wn = np.linalg.norm(synth.bf16_bits_to_f32(Wb).astype(np.float64) * M, axis=1)
    bound = np.outer(xn, wn) * 2.0 ** -14
    if bf16_out:
        bound += np.abs(want) * 2.0 ** -8
    else:
        bound += np.abs(want) * 2.0 ** -20
    bad = np.abs(got - want) > bound
    if bad.any():
        b, o = np.argwhere(bad)[0]
        raise AssertionError("%s: %d elements outside the bound, first at [%d, %d]: got %r want %r"
                             % (what, int(bad.sum()), b, o, got[b, o], want[b, o]))


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
        M = self.mask()
        return oracle.masked_gemm(self.Wb, M, self.Xb)

    def mask(self):
        return oracle.decode_mask(self.Ip, self.Iz, self.layer.rows, self.layer.cols)

    def check_full(self, algo, want=None, dtypes=(torch.bfloat16, torch.float32)):
        """Whole Y against the oracle: the Frobenius gate plus the per-element bound."""
        M = self.mask()
        want = oracle.masked_gemm(self.Wb, M, self.Xb) if want is None else want
        for dt in dtypes:
            got = self.run(algo, dt)
            bf = dt == torch.bfloat16
            assert rel_fro(got, want) <= (TOL if bf else TOL_F32), (dt, rel_fro(got, want))
            assert_elementwise(got, want, self.Xb, self.Wb, M, bf, str(dt))
        return want

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
    c = Case(synth.CONFIGS["alexnet_fc"], batch)
    c.check_full(b.ALGO_AUTO)


@pytest.mark.parametrize("shape", [
    # layer, batch: kernels whose ring of stages has an odd length (3 and 5) and whose K is split; a few-row pair layer
    ("alexnet_fc", 128), ("alexnet_fc", 16), ("conv3x3_256", 3136),
], ids=lambda s: "%s-%d" % s)
def test_repeated_launches_give_the_same_bits(shape):
    """The kernels are deterministic: 300 launches of one call must agree bit for bit with the first (checked against
    the oracle by the tests around this one).  A hand-over in the pipeline that is wrong only for some timings shows
    up here as a launch that differs."""
    b = _b()
    name, batch = shape
    L = synth.CONFIGS[name]
    c = Case(L, batch)
    first = b.lrbi_masked_gemm(L, c.W, c.ip, c.iz, c.X, y_dtype=torch.float32).clone()
    Y = torch.empty_like(first)
    differing = 0
    for _ in range(300):
        b.lrbi_masked_gemm(L, c.W, c.ip, c.iz, c.X, Y=Y, y_dtype=torch.float32)
        differing += int(not torch.equal(Y, first))
    torch.cuda.synchronize()
    assert differing == 0 and b.device_status() == 0


def test_conv3x3_config():
    b = _b()
    L = synth.CONFIGS["conv3x3_256"]
    c = Case(L, 12544)
    c.check_full(b.ALGO_AUTO, dtypes=(torch.bfloat16,))
    # property that holds at any size: a column of Y whose mask row is empty is exactly zero
    M = c.mask()
    empty_rows = np.flatnonzero(M.sum(axis=1) == 0)
    assert not c.run(b.ALGO_AUTO)[:, empty_rows].any()


def test_ffn_config_full():
    """The headline configuration, every one of its 67 M outputs (the oracle takes most of a minute)."""
    b = _b()
    L = synth.CONFIGS["ffn_16384x4096"]
    c = Case(L, 4096)
    plan = b.masked_gemm_plan(L, 4096)
    assert plan.algo == b.ALGO_TENSOR and plan.cta_pair == 1 and plan.k_splits == 1
    c.check_full(b.ALGO_AUTO, dtypes=(torch.bfloat16,))
    got = c.run(b.ALGO_AUTO)
    # linearity in X: doubling the activations doubles Y exactly (power of two scaling is exact in bf16/fp32)
    c.Xb = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(c.Xb) * np.float32(2.0))
    c.X = b.to_device_bf16(c.Xb)
    got2 = c.run(b.ALGO_AUTO)
    assert (got2[:64] == 2.0 * got[:64]).all()


# ------------------------------------------------------------------------------------------------
# CTA-pair instantiations of the tensor-core kernel (the ones large layers run on), with one accumulator
# (256 batch rows per pair, or 192: the tile of layers with few rows and a long batch) and with two (512 batch
# rows per pair; the headline workload's kernel).  They are forced through LRBI_ALGO_TENSOR_PAIR / _PAIR192 /
# _PAIR2 so that every shape below runs in all three; the shapes are
# wide in the batch and thin in K (the oracle stays under a second each).
# ------------------------------------------------------------------------------------------------
PAIR_SHAPES = [
    # rows, cols, tm, tn, k, batch
    (600, 320, 600, 320, 33, 9477),      # one tile; rows = 2*256 + 88: the second CTA of the last pair has no rows;
                                         # a 256-column panel followed by a ragged 64-column one; two index words
    (712, 384, 128, 128, 16, 9300),      # 128-column tiles: 64-column panels; rows = 2*256 + 200; batch tail of 84
    (512, 200, 128, 64, 145, 14200),     # 64-column tiles, last one ragged (8 columns); rank 145: five index words
    (512, 320, 256, 320, 256, 14300),    # rank 256: eight index words
    (1024, 512, 512, 256, 64, 7200),     # exact tiling in rows and K, ragged batch only
    (1000, 264, 1000, 264, 7, 7300),     # one tile, K = 4 blocks + 8 columns, rows tail of 232
    (384, 1344, 128, 1344, 40, 700),     # five full panels and one of 64 columns: both decoder groups, odd panel count
    (256, 2304, 128, 256, 16, 130),      # nine panels, batch just above one CTA's half of a 256-row accumulator
]


def _pair_algos():
    b = _b()
    return [(b.ALGO_TENSOR_PAIR, 256), (b.ALGO_TENSOR_PAIR2, 512), (b.ALGO_TENSOR_PAIR192, 192)]


@pytest.mark.parametrize("width", [192, 256, 512])
@pytest.mark.parametrize("shape", PAIR_SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_cta_pair_kernel(shape, width):
    b = _b()
    algo = dict((w, a) for a, w in _pair_algos())[width]
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("pair", rows, cols, tm, tn, k, 0.25, 0.05)
    plan = b.masked_gemm_plan(L, batch, algo)
    assert plan.cta_pair == 1 and plan.batch_tile == width
    assert plan.panel_columns == (256 if (L.grid[1] == 1 or L.tile_cols % 256 == 0) else 64)
    c = Case(L, batch)
    before = b.launch_count()
    c.check_full(algo)                                # bf16 and fp32 output
    assert b.launch_count() - before == 2 * (1 if plan.k_splits == 1 else 2)


def test_auto_choice_reaches_every_pair_instantiation():
    """What LRBI_ALGO_TENSOR picks by itself: pairs above 128 batch rows, two accumulators above 256, and 192-row
    tiles when those fit the chip in one wave (few rows, long batch)."""
    b = _b()
    L = synth.Layer("few", 256, 576, 128, 64, 16, 0.25, 0.05)
    plan = b.masked_gemm_plan(L, 1500, b.ALGO_TENSOR)
    assert plan.cta_pair == 1 and plan.batch_tile == 192
    Case(L, 1500).check_full(b.ALGO_TENSOR)
    L = synth.Layer("pair", 1024, 512, 512, 256, 64, 0.25, 0.05)
    for batch, width in ((200, 256), (7200, 512)):
        plan = b.masked_gemm_plan(L, batch, b.ALGO_TENSOR)
        assert plan.cta_pair == 1 and plan.batch_tile == width
        Case(L, batch).check_full(b.ALGO_TENSOR)
    # few output tiles and a long reduction: K is split in pair mode too (fp32 partial sums, second kernel)
    L = synth.Layer("pairsplit", 512, 4096, 256, 1024, 64, 0.25, 0.05)
    plan = b.masked_gemm_plan(L, 300, b.ALGO_TENSOR)
    assert plan.cta_pair == 1 and plan.k_splits > 1
    Case(L, 300).check_full(b.ALGO_TENSOR)


@pytest.mark.parametrize("width", [192, 256, 512])
def test_cta_pair_kernel_one_hot_and_degenerate_masks(width):
    b = _b()
    algo = dict((w, a) for a, w in _pair_algos())[width]
    shape = (712, 384, 128, 128, 16, 9300)
    rows, cols, tm, tn, k, batch = shape
    L = synth.Layer("pair", rows, cols, tm, tn, k, 0.25, 0.05)
    # one-hot activations return masked columns of W exactly
    c = Case(L, batch)
    cols_hit = (np.arange(batch) * 7 + 3) % L.cols
    X = np.zeros((batch, L.cols), dtype=np.float32)
    X[np.arange(batch), cols_hit] = 1.0
    c.Xb = synth.f32_to_bf16_bits(X)
    c.X = b.to_device_bf16(c.Xb)
    M = c.mask()
    want = (synth.bf16_bits_to_f32(c.Wb) * M)[:, cols_hit].T.astype(np.float64)
    assert (c.run(algo) == want).all()
    assert (c.run(algo, torch.float32) == want).all()
    # nothing kept / everything kept
    c = Case(L, batch, p=0.0)
    assert not c.run(algo).any()
    c = Case(L, batch, p=1.0)
    W = synth.bf16_bits_to_f32(c.Wb).astype(np.float64)
    Xf = synth.bf16_bits_to_f32(c.Xb).astype(np.float64)
    assert rel_fro(c.run(algo, torch.float32), Xf @ W.T) <= TOL_F32
    # NaN / Inf parked in pruned weights never reach Y
    c = Case(L, batch)
    M = c.mask()
    want = c.oracle_full()
    Wb = c.Wb.copy()
    Wb[M == 0] = np.where(np.arange((M == 0).sum()) % 2 == 0, 0x7FC0, 0xFF80).astype(np.uint16)
    c.Wb, c.W = Wb, b.to_device_bf16(Wb)
    got = c.run(algo)
    assert np.isfinite(got).all() and rel_fro(got, want) <= TOL


@pytest.mark.parametrize("k", [5, 33])
def test_bits_beyond_rank_are_ignored_by_every_gemm_kernel(k):
    """Garbage in bits >= k of the last packed word of both factors changes nothing."""
    b = _b()
    L = synth.Layer("pad", 256, 512, 128, 128, k, 0.25, 0.05)
    garbage = np.uint32((0xFFFFFFFF << (k % 32)) & 0xFFFFFFFF)
    for batch, algos in ((4, (b.ALGO_GENERIC, b.ALGO_GEMV, b.ALGO_STREAM)), (40, (b.ALGO_TENSOR,)), (300, (b.ALGO_TENSOR, b.ALGO_TENSOR_PAIR, b.ALGO_TENSOR_PAIR2, b.ALGO_TENSOR_PAIR192))):
        c = Case(L, batch)
        want = c.oracle_full()
        ipw, izw = synth.pack_ip(c.Ip).reshape(-1, L.kw), synth.pack_iz(c.Iz).reshape(-1, L.kw)
        ipw[:, -1] |= garbage
        izw[:, -1] |= garbage
        c.ip, c.iz = b.to_device_words(ipw.reshape(-1)), b.to_device_words(izw.reshape(-1))
        for algo in algos:
            assert rel_fro(c.run(algo, torch.float32), want) <= TOL_F32, b.ALGO_NAMES[algo]
