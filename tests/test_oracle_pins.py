"""Pins for the CPU oracle: everything it is compared with here comes from the paper's
printed example, from brute force, from closed forms or from a library routine -- never
from the oracle itself and never from the CUDA path."""
import itertools
import os

import numpy as np
import pytest

import oracle
from conftest import GOLDEN, read_golden_matrices
from paper_1905_05686_b200 import synth

G = read_golden_matrices(os.path.join(GOLDEN, "worked_example.txt"))


def untiled(decode, Ip, Iz):
    """Call a decode function on one tile equal to the matrix."""
    m, _ = Ip.shape
    _, n = Iz.shape
    return decode(Ip[None, None], Iz[None, None], m, n)


def or_of_outer_products(Ip, Iz):
    """Independent formulation of Eq. 3: Ia = OR over l of (column l of Ip) x (row l of Iz)."""
    out = np.zeros((Ip.shape[0], Iz.shape[1]), dtype=bool)
    for l in range(Ip.shape[1]):
        out |= np.outer(Ip[:, l].astype(bool), Iz[l, :].astype(bool))
    return out.astype(np.uint8)


# --------------------------------------------------------------------------- decode pins
def pin_worked_example(decode):
    Ip, Iz = G["Ip"].astype(np.uint8), G["Iz"].astype(np.uint8)
    Ia = untiled(decode, Ip, Iz)
    assert (Ia == G["Ia"]).all()
    diff = np.argwhere(Ia != G["I"]) + 1  # 1-based, as in the text under Eq. 6
    assert sorted(map(tuple, diff)) == [(1, 5), (3, 3)]


def pin_bruteforce_tiny(decode):
    # every Ip (2xk), Iz (kx3) for k = 1, 2: 2^(2k) * 2^(3k) cases
    for k in (1, 2):
        for bits in itertools.product((0, 1), repeat=2 * k + 3 * k):
            Ip = np.array(bits[: 2 * k], dtype=np.uint8).reshape(2, k)
            Iz = np.array(bits[2 * k:], dtype=np.uint8).reshape(k, 3)
            exp = np.zeros((2, 3), dtype=np.uint8)
            for i in range(2):
                for j in range(3):
                    exp[i, j] = int(any(Ip[i, l] and Iz[l, j] for l in range(k)))
            assert (untiled(decode, Ip, Iz) == exp).all()


def pin_random_vs_outer_products(decode):
    rng = np.random.default_rng(7)
    for m, n, k in [(3, 9, 4), (9, 3, 7), (5, 8, 1), (7, 7, 33), (4, 6, 70)]:
        Ip = (rng.random((m, k)) < 0.3).astype(np.uint8)
        Iz = (rng.random((k, n)) < 0.3).astype(np.uint8)
        assert (untiled(decode, Ip, Iz) == or_of_outer_products(Ip, Iz)).all()


def pin_identity(decode):
    rng = np.random.default_rng(3)
    Mx = (rng.random((6, 11)) < 0.4).astype(np.uint8)
    assert (untiled(decode, np.eye(6, dtype=np.uint8), Mx) == Mx).all()       # Ip = I  ->  Ia = Iz
    assert (untiled(decode, Mx, np.eye(11, dtype=np.uint8)) == Mx).all()      # Iz = I  ->  Ia = Ip


def pin_rank_one_and_transpose(decode):
    rng = np.random.default_rng(5)
    u = (rng.random((7, 1)) < 0.5).astype(np.uint8)
    v = (rng.random((1, 9)) < 0.5).astype(np.uint8)
    assert (untiled(decode, u, v) == u * v).all()
    Ip = (rng.random((6, 5)) < 0.3).astype(np.uint8)
    Iz = (rng.random((5, 8)) < 0.3).astype(np.uint8)
    assert (untiled(decode, Ip, Iz).T == untiled(decode, Iz.T.copy(), Ip.T.copy())).all()


def pin_tiling(decode):
    rng = np.random.default_rng(11)
    rows, cols, tm, tn, k = 10, 14, 4, 5, 3          # ragged: 3x3 grid, last tiles cut
    gr, gc = 3, 3
    Ip = (rng.random((gr, gc, tm, k)) < 0.4).astype(np.uint8)
    Iz = (rng.random((gr, gc, k, tn)) < 0.4).astype(np.uint8)
    M = decode(Ip, Iz, rows, cols)
    assert M.shape == (rows, cols)
    for tr in range(gr):
        for tc in range(gc):
            blk = or_of_outer_products(Ip[tr, tc], Iz[tr, tc])
            r0, c0 = tr * tm, tc * tn
            sub = M[r0:r0 + tm, c0:c0 + tn]
            assert (sub == blk[: sub.shape[0], : sub.shape[1]]).all()


DECODE_PINS = [pin_worked_example, pin_bruteforce_tiny, pin_random_vs_outer_products,
               pin_identity, pin_rank_one_and_transpose, pin_tiling]


@pytest.mark.parametrize("pin", DECODE_PINS, ids=lambda f: f.__name__)
def test_decode_pin(pin):
    pin(oracle.decode_mask)


# Plausible mistakes, planted in CPU stand-ins: each must be caught by at least one pin.
def _mut_and_or_swapped(Ip, Iz, rows, cols):            # AND of ORs instead of OR of ANDs
    return _mut_generic(Ip, Iz, rows, cols, lambda a, b: np.all(a | b))


def _mut_drop_last_term(Ip, Iz, rows, cols):            # loop stops at k-1
    return _mut_generic(Ip, Iz, rows, cols, lambda a, b: np.any(a[:-1] & b[:-1]) if len(a) > 1 else np.any(a & b))


def _mut_xor(Ip, Iz, rows, cols):                        # GF(2) product instead of Boolean
    return _mut_generic(Ip, Iz, rows, cols, lambda a, b: np.sum(a & b) % 2)


def _mut_generic(Ip, Iz, rows, cols, f, tile_swap=False):
    gr, gc, tm, k = Ip.shape
    tn = Iz.shape[3]
    M = np.zeros((rows, cols), dtype=np.uint8)
    for r in range(rows):
        for c in range(cols):
            tr, tc = r // tm, c // tn
            if tile_swap and tr < gc and tc < gr:
                tr, tc = tc, tr
            M[r, c] = int(f(Ip[tr, tc, r % tm, :], Iz[tr, tc, :, c % tn]))
    return M


def _mut_tile_index_transposed(Ip, Iz, rows, cols):      # tile (tr, tc) read as (tc, tr)
    return _mut_generic(Ip, Iz, rows, cols, lambda a, b: np.any(a & b), tile_swap=True)


def _mut_correct(Ip, Iz, rows, cols):
    return _mut_generic(Ip, Iz, rows, cols, lambda a, b: np.any(a & b))


@pytest.mark.parametrize("mutant", [_mut_and_or_swapped, _mut_drop_last_term, _mut_xor, _mut_tile_index_transposed],
                         ids=lambda f: f.__name__)
def test_decode_pins_catch_planted_mistakes(mutant):
    caught = []
    for pin in DECODE_PINS:
        try:
            pin(mutant)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, "no pin notices this mistake"
    for pin in DECODE_PINS:                                # and the pins accept a correct stand-in
        pin(_mut_correct)


def test_monotone_in_factor_bits():
    L = synth.Layer("mono", 40, 70, 16, 32, 5, 0.2)
    Ip, Iz = synth.make_factors(L)
    base = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    Ip2 = Ip.copy()
    Ip2[1, 2, 3, 4] = 1
    assert (oracle.decode_mask(Ip2, Iz, L.rows, L.cols) >= base).all()


def test_density_matches_bit_count_and_eq7():
    L = synth.CONFIGS["decode_4096"]
    Ip, Iz = synth.make_factors(L)
    M = oracle.decode_mask(Ip, Iz, L.rows, L.cols)
    assert synth.popcount_words(synth.pack_mask(M)) == int(M.sum(dtype=np.int64))
    # Eq. 7 with S_p = S_z = 1 - p: expected density 1 - (1 - p^2)^k = d (mean only; bits are correlated)
    assert abs(M.mean() - L.density) < 3e-3
    # one tile in full against the independent formulation
    blk = or_of_outer_products(Ip[3, 5], Iz[3, 5])
    assert (M[3 * 256:4 * 256, 5 * 256:6 * 256] == blk).all()


# --------------------------------------------------------------------------- storage pins
def _golden_sizes():
    out = {}
    with open(os.path.join(GOLDEN, "storage_sizes.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                p = line.split()
                out[p[0]] = float(p[1])
    return out


def test_packed_factor_bytes_match_paper_tables():
    S = _golden_sizes()
    fc1 = synth.CONFIGS["lenet_fc1"]
    Ip, Iz = synth.make_factors(fc1)
    nbytes = (synth.pack_ip(Ip).size + synth.pack_iz(Iz).size) * 4
    # k = 16 occupies half of each 32-bit word: the information content is k(m+n)/8 bytes
    assert nbytes * fc1.rank // 32 == fc1.index_bytes == round(S["fc1_proposed_k16"] * 1000)
    assert fc1.mask_words * 4 == round(S["fc1_binary_index"] * 1000)
    fc6 = synth.Layer("fc6", 4096, 4096, 512, 512, 32, 0.09)
    assert fc6.grid == (8, 8)
    Ip, Iz = synth.make_factors(fc6)
    assert (synth.pack_ip(Ip).size + synth.pack_iz(Iz).size) * 4 == S["fc6_proposed_k32"] * 1024
    assert fc6.mask_words * 4 == S["fc6_binary_index"] * 1024
    for k in (4, 8, 16, 32, 64, 128, 256):
        assert round(500 * 800 / (k * (500 + 800)), 1) == S["ratio_k%d" % k]


def test_pack_roundtrip_and_bit_order():
    Ip = np.zeros((1, 1, 3, 40), dtype=np.uint8)
    Ip[0, 0, 1, 0] = 1
    Ip[0, 0, 1, 33] = 1
    Ip[0, 0, 2, 31] = 1
    w = synth.pack_ip(Ip).reshape(3, 2)
    assert w.tolist() == [[0, 0], [1, 2], [1 << 31, 0]]
    Iz = np.zeros((1, 1, 40, 2), dtype=np.uint8)
    Iz[0, 0, 35, 1] = 1
    assert synth.pack_iz(Iz).reshape(2, 2).tolist() == [[0, 0], [0, 8]]
    rng = np.random.default_rng(0)
    M = (rng.random((5, 77)) < 0.5).astype(np.uint8)
    pm = synth.pack_mask(M)
    assert pm.shape == (5, 3) and (synth.unpack_mask(pm, 77) == M).all()
    assert (pm[:, 2] >> 13 == 0).all()                    # pad bits are zero


# --------------------------------------------------------------------------- masked GEMM pins
def test_threshold_steps_of_worked_example():
    # Eq. 1 -> Eq. 2 (|w| >= 0.7) and Eq. 4 -> Eq. 5 (>= T_p, >= T_z): fixes polarity 1 = kept
    assert ((np.abs(G["W"]) >= 0.7) == G["I"]).all()
    assert ((G["Mp"] >= 0.5) == G["Ip"]).all() and ((G["Mz"] >= 0.6) == G["Iz"]).all()


def test_masked_gemm_worked_example_by_hand():
    Wb = synth.f32_to_bf16_bits(G["W"].astype(np.float32))
    X = np.eye(5, dtype=np.float32)
    X = np.vstack([X, np.ones((1, 5), dtype=np.float32)])
    Y = oracle.masked_gemm(Wb, G["I"].astype(np.uint8), synth.f32_to_bf16_bits(X))
    # row sums of W .* I worked out by hand from Eq. 1 and Eq. 2
    by_hand = np.array([0.9 + 1.2, 1.8 - 0.7 - 1.6, -1.7 + 1.2, 1.4 - 0.9 + 1.4, -1.1 + 1.0 + 1.0])
    assert np.abs(Y[5] - by_hand).max() < 5 * 2.0**-8 * 1.8
    # one-hot rows of X pick out columns of (W .* I)^T exactly (bf16 values, no rounding)
    Wm = synth.bf16_bits_to_f32(Wb).astype(np.float64) * G["I"]
    assert (Y[:5] == Wm.T).all()


def test_masked_gemm_special_cases_against_numpy():
    rng = np.random.default_rng(1)
    N, K, B = 37, 53, 9
    Wb = synth.f32_to_bf16_bits(rng.standard_normal((N, K), dtype=np.float32))
    Xb = synth.f32_to_bf16_bits(rng.standard_normal((B, K), dtype=np.float32))
    W = synth.bf16_bits_to_f32(Wb).astype(np.float64)
    X = synth.bf16_bits_to_f32(Xb).astype(np.float64)
    assert (oracle.bf16_to_f64(Wb) == W).all()
    ones = np.ones((N, K), dtype=np.uint8)
    np.testing.assert_allclose(oracle.masked_gemm(Wb, ones, Xb), X @ W.T, rtol=0, atol=1e-12)
    assert (oracle.masked_gemm(Wb, np.zeros_like(ones), Xb) == 0).all()
    M = (rng.random((N, K)) < 0.3).astype(np.uint8)
    np.testing.assert_allclose(oracle.masked_gemm(Wb, M, Xb), X @ (W * M).T, rtol=0, atol=1e-12)
    # transposed-operand mistake would show here: N != K != B
    # select, not multiply: a NaN stored in a pruned weight must not reach Y
    Wb2 = Wb.copy()
    Wb2[M == 0] = 0x7FC0
    np.testing.assert_allclose(oracle.masked_gemm(Wb2, M, Xb), X @ (W * M).T, rtol=0, atol=1e-12)


def test_samples_agree_with_definition_by_parts():
    L = synth.Layer("s", 45, 100, 16, 32, 9, 0.25)
    Ip, Iz = synth.make_factors(L)
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, 6)
    W = synth.bf16_bits_to_f32(Wb).astype(np.float64)
    X = synth.bf16_bits_to_f32(Xb).astype(np.float64)
    gr, gc = L.grid
    M = np.zeros((gr * 16, gc * 32), dtype=np.uint8)
    for tr in range(gr):
        for tc in range(gc):
            M[tr * 16:(tr + 1) * 16, tc * 32:(tc + 1) * 32] = or_of_outer_products(Ip[tr, tc], Iz[tr, tc])
    M = M[:45, :100]
    full = X @ (W * M).T
    b_idx = np.array([0, 5, 3, 2, 1, 4, 0], dtype=np.int64)
    o_idx = np.array([0, 44, 17, 31, 16, 15, 32], dtype=np.int64)
    got = oracle.masked_gemm_samples(Wb, Ip, Iz, Xb, b_idx, o_idx)
    np.testing.assert_allclose(got, full[b_idx, o_idx], rtol=0, atol=1e-12)


def test_generator_is_seeded_and_shaped():
    L = synth.CONFIGS["lenet_fc1"]
    a, b = synth.make_factors(L)
    a2, b2 = synth.make_factors(L)
    assert (a == a2).all() and (b == b2).all() and a.shape == (1, 1, 500, 16) and b.shape == (1, 1, 16, 800)
    assert abs(a.mean() - L.p) < 0.01 and abs(b.mean() - L.p) < 0.01
    w = synth.bf16_bits_to_f32(synth.make_weights(L))
    assert abs(w.std() - 0.05) < 1e-3 and abs(w.mean()) < 1e-3
    # bf16 rounding: nearest, ties to even
    x = np.array([1.0, 1.00390625, 1.01171875, -1.00390625], dtype=np.float32)   # 1, 1+2^-8 (tie), 1+3*2^-8 (tie), ...
    assert synth.f32_to_bf16_bits(x).tolist() == [0x3F80, 0x3F80, 0x3F82, 0xBF80]


# --------------------------------------------------------------------------- one rank per tile
def test_decode_with_one_rank_per_tile():
    """Section 3.1, last paragraph.  Pinned by what it must reduce to: every tile decoded on its own, untiled,
    from the first ranks[t] columns/rows of its factors (OR of outer products); equal ranks give the plain
    tiled decode; what lies beyond a tile's rank changes nothing; rank 0 gives an empty tile."""
    rng = np.random.default_rng(21)
    rows, cols, tm, tn, kmax = 11, 13, 4, 5, 6
    gr, gc = -(-rows // tm), -(-cols // tn)
    Ip = (rng.random((gr, gc, tm, kmax)) < 0.35).astype(np.uint8)
    Iz = (rng.random((gr, gc, kmax, tn)) < 0.35).astype(np.uint8)
    ranks = rng.integers(0, kmax + 1, gr * gc).astype(np.int32)
    ranks[0], ranks[1] = 0, kmax
    M = oracle.decode_mask_ranks(Ip, Iz, ranks, rows, cols)
    for tr in range(gr):
        for tc in range(gc):
            k = ranks[tr * gc + tc]
            want = or_of_outer_products(Ip[tr, tc][:, :k], Iz[tr, tc][:k, :]) if k else np.zeros((tm, tn), np.uint8)
            blk = M[tr * tm:(tr + 1) * tm, tc * tn:(tc + 1) * tn]
            assert (blk == want[:blk.shape[0], :blk.shape[1]]).all()
    assert not M[:tm, :tn].any()                                           # rank 0
    full = np.full(gr * gc, kmax, dtype=np.int32)
    assert (oracle.decode_mask_ranks(Ip, Iz, full, rows, cols) == oracle.decode_mask(Ip, Iz, rows, cols)).all()
    Ip2, Iz2 = Ip.copy(), Iz.copy()
    for t in range(gr * gc):                                               # garbage beyond each tile's rank
        Ip2.reshape(gr * gc, tm, kmax)[t][:, ranks[t]:] = 1
        Iz2.reshape(gr * gc, kmax, tn)[t][ranks[t]:, :] = 1
    assert (oracle.decode_mask_ranks(Ip2, Iz2, ranks, rows, cols) == M).all()


# --------------------------------------------------------------------------- masked backward
def test_masked_backward():
    """Pinned by numpy's fp64 matmul on the masked weights, by the adjoint identities that tie it to the (separately
    pinned) forward product, and by the special masks: full mask = the plain GEMM gradients, empty mask = zeros."""
    rng = np.random.default_rng(9)
    B, N, K = 5, 7, 11
    bits = lambda a: synth.f32_to_bf16_bits(a.astype(np.float32))
    Wb, Xb, dYb = bits(rng.standard_normal((N, K))), bits(rng.standard_normal((B, K))), bits(rng.standard_normal((B, N)))
    f = lambda b: synth.bf16_bits_to_f32(b).astype(np.float64)
    for M in (np.ones((N, K), np.uint8), np.zeros((N, K), np.uint8), (rng.random((N, K)) < 0.4).astype(np.uint8)):
        dX, dW = oracle.masked_backward(Wb, M, Xb, dYb)
        assert np.allclose(dX, f(dYb) @ (f(Wb) * M), rtol=1e-12, atol=1e-12)       # [B,N] x [N,K]
        assert np.allclose(dW, (f(dYb).T @ f(Xb)) * M, rtol=1e-12, atol=1e-12)     # ([N,B] x [B,K]) .* M
        assert not dW[M == 0].any()
        # <dY, Y(E)> = <dX, E> for any activations E, and <dY, Y with weights F> = <dW, F> for any weights F
        Eb, Fb = bits(rng.standard_normal((B, K))), bits(rng.standard_normal((N, K)))
        assert np.sum(f(dYb) * oracle.masked_gemm(Wb, M, Eb)) == pytest.approx(np.sum(dX * f(Eb)), rel=1e-10, abs=1e-10)
        assert np.sum(f(dYb) * oracle.masked_gemm(Fb, M, Xb)) == pytest.approx(np.sum(dW * f(Fb)), rel=1e-10, abs=1e-10)
    # a transposed operand would fail the shapes above (B, N, K all differ); a NaN in a pruned weight reaches neither
    M = (rng.random((N, K)) < 0.5).astype(np.uint8)
    Wn = Wb.copy()
    Wn[M == 0] = 0x7FC0
    assert np.array_equal(oracle.masked_backward(Wn, M, Xb, dYb)[0], oracle.masked_backward(Wb, M, Xb, dYb)[0])
