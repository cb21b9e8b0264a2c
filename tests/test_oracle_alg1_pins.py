"""Pins for the oracle of Algorithm 1's inner loop (binary conversion, sparsity, cost, the S_p sweep).

Expected values come from the paper's printed example (Eq. 1, 2, 4, 5, 6 and the sentence under Eq. 6),
from closed forms, from vectorised numpy on random inputs and from exhaustive enumeration on a tiny
case -- never from the oracle itself and never from the CUDA path."""
import itertools
import os

import numpy as np
import pytest

import oracle
from conftest import GOLDEN, read_golden_matrices
from paper_1905_05686_b200 import synth

G = read_golden_matrices(os.path.join(GOLDEN, "worked_example.txt"))
# bf16 keeps 8 significant bits: 0.7 becomes 0.69921875, so the example's threshold is rounded the same way
# (|-0.7| must still count as "not below the threshold", as it does in Eq. 2)
W_BITS = synth.f32_to_bf16_bits(G["W"].astype(np.float32))
THETA = float(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(np.array([0.7], dtype=np.float32)))[0])


def test_binary_conversion_reproduces_eq5_from_eq4():
    Mp, Mz = G["Mp"].astype(np.float32)[None], G["Mz"].astype(np.float32)[None]
    assert (oracle.threshold(Mp, 0.5)[0] == G["Ip"]).all()        # T_p = 0.5: the entry 0.5 itself becomes 1 (">=")
    assert (oracle.threshold(Mz, 0.6)[0] == G["Iz"]).all()        # T_z = 0.6
    assert oracle.threshold(Mp, np.nextafter(np.float32(0.5), np.float32(1)))[0][0, 1] == 0   # a strict ">" would differ here


def test_threshold_is_per_tile():
    v = np.array([[0.1, 0.4, 0.9], [0.1, 0.4, 0.9]], dtype=np.float32)
    got = oracle.threshold(v, np.array([0.4, 0.5], dtype=np.float32))
    assert got.tolist() == [[0, 1, 1], [0, 0, 1]]
    assert oracle.threshold(v, np.float32(np.inf)).sum() == 0 and oracle.threshold(v, 0.0).sum() == 6


def test_index_and_cost_on_the_papers_example():
    """Eq. 1 with threshold 0.7 gives Eq. 2 (13 ones, S = 12/25); Eq. 6 has 15 ones (S_a = 10/25); its two
    mismatches are ones of Ia where I is 0, so no kept weight is lost and the cost is 0."""
    kept_i, kept_a, lost, cost = oracle.index_cost(W_BITS, THETA, G["Ia"].astype(np.uint8), 5, 5)
    assert (kept_i[0], kept_a[0], lost[0], cost[0]) == (13, 15, 0, 0.0)
    # I itself as the decoded index: nothing lost either; an empty index loses every kept weight
    I = G["I"].astype(np.uint8)
    assert oracle.index_cost(W_BITS, THETA, I, 5, 5)[2][0] == 0
    kept_i, kept_a, lost, cost = oracle.index_cost(W_BITS, THETA, np.zeros((5, 5), np.uint8), 5, 5)
    by_hand = sum(abs(float(v)) for v, keep in zip(synth.bf16_bits_to_f32(W_BITS).ravel(), I.ravel()) if keep)
    assert (kept_a[0], lost[0]) == (0, 13) and cost[0] == pytest.approx(by_hand, rel=1e-12)
    # dropping exactly one kept position, (2, 1) with |W| = 1.8 (0-based (1, 0)), costs exactly that weight
    Ia = G["Ia"].astype(np.uint8).copy()
    Ia[1, 0] = 0
    _, _, lost, cost = oracle.index_cost(W_BITS, THETA, Ia, 5, 5)
    assert lost[0] == 1 and cost[0] == float(synth.bf16_bits_to_f32(W_BITS)[1, 0])


def test_index_cost_against_numpy_on_random_tiled_layers():
    rng = np.random.default_rng(11)
    for rows, cols, tm, tn in [(7, 9, 7, 9), (10, 12, 4, 5), (33, 70, 16, 32), (5, 5, 2, 2)]:
        Wb = synth.f32_to_bf16_bits(rng.standard_normal((rows, cols)).astype(np.float32))
        Ia = (rng.random((rows, cols)) < 0.4).astype(np.uint8)
        theta = 0.8
        kept_i, kept_a, lost, cost = oracle.index_cost(Wb, theta, Ia, tm, tn)
        A = np.abs(synth.bf16_bits_to_f32(Wb).astype(np.float64))
        I = A >= np.float64(np.float32(theta))
        gr, gc = -(-rows // tm), -(-cols // tn)
        for tr in range(gr):
            for tc in range(gc):
                sl = (slice(tr * tm, (tr + 1) * tm), slice(tc * tn, (tc + 1) * tn))
                t = tr * gc + tc
                assert kept_i[t] == I[sl].sum() and kept_a[t] == Ia[sl].sum()
                miss = I[sl] & (Ia[sl] == 0)
                assert lost[t] == miss.sum()
                assert cost[t] == pytest.approx(A[sl][miss].sum(), rel=1e-12, abs=0)
        assert kept_i.sum() == I.sum()                           # tiles partition the matrix


def test_nan_weights_count_as_pruned():
    Wb = np.array([[0x7FC0, 0x3F80]], dtype=np.uint16)            # NaN, 1.0
    kept_i, _, lost, cost = oracle.index_cost(Wb, 0.5, np.zeros((1, 2), np.uint8), 1, 2)
    assert (kept_i[0], lost[0], cost[0]) == (1, 1, 1.0)


def test_eq7_inversion():
    for S, Sp, k in [(0.48, 0.5, 2), (0.9, 0.3, 16), (0.95, 0.0, 64)]:
        Sz = oracle.sz_from_eq7(S, Sp, k)
        assert (1 - (1 - Sp) * (1 - Sz)) ** k == pytest.approx(S, rel=1e-12)
    # equal factor sparsities 1 - p with p = sqrt(1 - (1 - d)^(1/k)): the generator's density formula
    d, k = 0.2, 64
    p = np.sqrt(1 - (1 - d) ** (1.0 / k))
    assert oracle.sz_from_eq7(1 - d, 1 - p, k) == pytest.approx(1 - p, rel=1e-9)
    assert oracle.sz_from_eq7(0.48, 0.5, 2) == pytest.approx((np.sqrt(0.48) - 0.5) / 0.5)


def test_threshold_for_sparsity():
    v = np.array([0.0, 0.0, 0.2, 0.2, 0.3, 0.5, 0.8, 0.8, 0.9, 1.3], dtype=np.float32)   # Mp of Eq. 4, sorted
    assert oracle.threshold_for_sparsity(v, 0.5) == np.float32(0.5)                      # five entries fall below 0.5
    assert oracle.threshold_for_sparsity(v, 0.0) == np.float32(0.0)
    assert np.isinf(oracle.threshold_for_sparsity(v, 1.0))
    t = oracle.threshold_for_sparsity(v, 0.3)                                            # three below: tie at 0.2 kept
    assert t == np.float32(0.2) and (v >= t).sum() == 8


def _cost_numpy(Wb, theta, Ip, Iz):
    A = np.abs(synth.bf16_bits_to_f32(Wb).astype(np.float64))
    I = A >= np.float64(np.float32(theta))
    Ia = (Ip.astype(np.int64) @ Iz.astype(np.int64)) > 0
    return float(A[I & ~Ia].sum()), 1.0 - Ia.mean()


def test_search_on_the_papers_example():
    r = oracle.alg1_search(W_BITS, THETA, G["Mp"], G["Mz"], sp_step=0.1, tol=0.05)
    assert r["S"] == pytest.approx(12 / 25)
    assert len(r["tried"]) == 11 and [c["Sp"] for c in r["tried"]] == pytest.approx([i / 10 for i in range(11)])
    assert r["best"]["cost"] == min(c["cost"] for c in r["tried"])
    first_min = next(c for c in r["tried"] if c["cost"] == r["best"]["cost"])
    assert first_min is r["best"]                                  # "if Cost_min > Cost": the first minimum is kept
    Mp, Mz = G["Mp"].astype(np.float32), G["Mz"].astype(np.float32)
    for c in r["tried"]:                                           # every candidate's numbers follow from its thresholds
        cost, Sa = _cost_numpy(W_BITS, THETA, Mp >= np.float32(c["Tp"]), Mz >= np.float32(c["Tz"]))
        assert c["cost"] == pytest.approx(cost, rel=1e-12, abs=0) and c["Sa"] == pytest.approx(Sa)
    half = next(c for c in r["tried"] if c["Sp"] == pytest.approx(0.5))
    assert half["Tp"] == 0.5                                       # S_p = 0.5 gives the paper's T_p and hence Eq. 5's Ip
    empty = r["tried"][-1]                                         # S_p = 1: Ip empty, every kept weight lost
    assert empty["lost"] == 13


def test_search_never_beats_exhaustive_enumeration():
    """On a tiny matrix every pair of thresholds can be tried: no pair that meets the sparsity tolerance costs
    more than ... nothing, the sweep is a heuristic; but it can never cost LESS than the best such pair."""
    rng = np.random.default_rng(5)
    m, n, k = 6, 7, 2
    Wb = synth.f32_to_bf16_bits(rng.standard_normal((m, n)).astype(np.float32))
    Mp, Mz = rng.random((m, k)).astype(np.float32), rng.random((k, n)).astype(np.float32)
    theta, tol = 0.6, 0.08
    r = oracle.alg1_search(Wb, theta, Mp, Mz, sp_step=0.1, tol=tol)
    S = r["S"]
    best = np.inf
    for tp, tz in itertools.product(list(np.unique(Mp)) + [np.inf], list(np.unique(Mz)) + [np.inf]):
        cost, Sa = _cost_numpy(Wb, theta, Mp >= tp, Mz >= tz)
        if abs(Sa - S) <= tol:
            best = min(best, cost)
    met = [c for c in r["tried"] if abs(c["Sa"] - S) <= tol]
    assert met, "no candidate of the sweep met the sparsity tolerance"
    assert min(c["cost"] for c in met) >= best - 1e-12


def test_planted_mistakes_are_caught():
    """Plausible mistakes in the cost (roles of I and Ia swapped; counting every mismatch) give other numbers on
    the paper's own example, so the pins above would catch them."""
    A = np.abs(synth.bf16_bits_to_f32(W_BITS).astype(np.float64))
    I, Ia = G["I"].astype(bool), G["Ia"].astype(bool)
    swapped = A[~I & Ia].sum()
    any_mismatch = A[I ^ Ia].sum()
    assert swapped > 0 and any_mismatch > 0                        # the oracle's 0.0 is not what these would give


# --------------------------------------------------------------------------- NMF by multiplicative updates
def _bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_nmf_one_step_by_hand():
    """M = [[1, 2], [2, 4]] from Mp = (1, 1)^T, Mz = (1, 1): Mz becomes (3, 6) / 2 = (1.5, 3), then Mp becomes
    (7.5, 15) / 11.25 = (2/3, 4/3), and Mp Mz is M exactly: a rank-one matrix is recovered in one iteration."""
    Mp, Mz = oracle.nmf_multiplicative(_bits([[1, -2], [2, 4]]), np.ones((1, 2, 1)), np.ones((1, 1, 2)), 2, 2, 1, eps=0.0)
    assert Mz[0].tolist() == [[1.5, 3.0]]
    assert Mp[0][:, 0] == pytest.approx([2 / 3, 4 / 3], rel=1e-15)
    assert (Mp[0] @ Mz[0]) == pytest.approx(np.array([[1, 2], [2, 4.0]]), rel=1e-15)          # |W| is factorised, not W


def test_nmf_properties():
    """Non-negative factors stay non-negative, the Frobenius objective never increases (the property the update rule
    is known for), an exact factorisation is a fixed point, and every tile is its own problem."""
    rng = np.random.default_rng(4)
    rows, cols, tm, tn, k = 12, 14, 6, 7, 3
    Wb = _bits(rng.standard_normal((rows, cols)))
    A = np.abs(synth.bf16_bits_to_f32(Wb).astype(np.float64))
    Mp0, Mz0 = rng.random((4, tm, k)) + 0.1, rng.random((4, k, tn)) + 0.1
    prev = None
    for it in range(0, 6):
        Mp, Mz = oracle.nmf_multiplicative(Wb, Mp0, Mz0, tm, tn, it)
        assert (Mp >= 0).all() and (Mz >= 0).all()
        err = sum(np.linalg.norm(A[tr * tm:(tr + 1) * tm, tc * tn:(tc + 1) * tn] - Mp[tr * 2 + tc] @ Mz[tr * 2 + tc]) ** 2
                  for tr in range(2) for tc in range(2))
        assert prev is None or err <= prev * (1 + 1e-12)
        prev = err
    # tile 3 alone, as a 6 x 7 matrix of its own, gives the same factors
    Mp1, Mz1 = oracle.nmf_multiplicative(Wb[6:, 7:], Mp0[3:], Mz0[3:], tm, tn, 5)
    assert np.allclose(Mp1[0], Mp[3], rtol=1e-13) and np.allclose(Mz1[0], Mz[3], rtol=1e-13)
    # exact factorisation: nothing moves (values chosen exactly representable in bf16)
    P = np.array([[1.0, 0.5], [2.0, 0.0], [0.25, 1.0]])
    Z = np.array([[1.0, 2.0, 0.5, 0.0], [0.5, 0.0, 1.0, 2.0]])
    Mp, Mz = oracle.nmf_multiplicative(_bits(P @ Z), P[None], Z[None], 3, 4, 3, eps=0.0)
    assert np.allclose(Mp[0], P, rtol=1e-14) and np.allclose(Mz[0], Z, rtol=1e-14)
    # ragged edge tiles: what lies outside the matrix counts as zero
    Mp, Mz = oracle.nmf_multiplicative(Wb[:9, :10], Mp0, Mz0, tm, tn, 2)
    pad = np.zeros((12, 14)); pad[:9, :10] = A[:9, :10]
    Mp2, Mz2 = oracle.nmf_multiplicative(_bits(pad), Mp0, Mz0, tm, tn, 2)
    assert np.allclose(Mp, Mp2) and np.allclose(Mz, Mz2)
