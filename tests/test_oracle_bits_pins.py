"""Pins of the oracle's rank-based bit-width assignment (CPU only): class counts, order
property, tie rule, brute-force ranks on small inputs, the library sort, and the counts the
adaptive benchmark configuration fixes (410 / 1228 / 3277 / 3277 of 8192 tokens)."""
import numpy as np
import pytest

import oracle
from golden_io import read_fixture
from rank_rule import by_library_sort
from paper_2605_03884_b200 import workloads as wl


def _cuts(T):
    c16 = int(np.floor(0.05 * T + 0.5)); c8 = int(np.floor(0.20 * T + 0.5)); c4 = int(np.floor(0.60 * T + 0.5))
    return c16, c8 - c16, c4 - c8


def test_counts_of_the_adaptive_configuration():
    T = 8192
    scores = np.random.default_rng(1007).lognormal(0.0, 1.0, size=T).astype(np.float32)
    n16, n8, n4 = _cuts(T)
    assert (n16, n8, n4, T - n16 - n8 - n4) == (410, 1228, 3277, 3277)
    st, bits = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == oracle.OK
    assert [(bits == b).sum() for b in (16, 8, 4, 2)] == [410, 1228, 3277, 3277]
    assert bits.astype(np.float64).mean() == pytest.approx(4.40, abs=0.005)


@pytest.mark.parametrize("T", [1, 2, 7, 64, 1000])
def test_higher_scores_never_get_fewer_bits_and_counts_hold(T):
    scores = np.random.default_rng(T).standard_normal(T).astype(np.float32)
    n16, n8, n4 = _cuts(T)
    st, bits = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == oracle.OK
    assert (bits == 16).sum() == n16 and (bits == 8).sum() == n8 and (bits == 4).sum() == n4
    order = np.argsort(-scores, kind="stable")
    assert np.all(np.diff(bits[order].astype(int)) <= 0)


def test_brute_force_rank_with_many_ties():
    T = 300
    scores = np.random.default_rng(5).integers(0, 6, size=T).astype(np.float32)   # six levels only
    n16, n8, n4 = 31, 77, 101
    st, bits = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == oracle.OK
    for t in range(T):
        rank = int((scores > scores[t]).sum() + (scores[:t] == scores[t]).sum())
        want = 16 if rank < n16 else 8 if rank < n16 + n8 else 4 if rank < n16 + n8 + n4 else 2
        assert bits[t] == want


def test_equal_scores_favour_the_lower_index():
    st, bits = oracle.bits_from_scores(np.zeros(10, np.float32), 2, 3, 1)
    assert st == oracle.OK and bits.tolist() == [16, 16, 8, 8, 8, 4, 2, 2, 2, 2]


def test_matches_the_library_sort():
    """The same rule stated with numpy's lexsort (score descending, index ascending), on random
    scores, on scores with many ties, and on the adaptive workload's own scores."""
    T = 4096
    n16, n8, n4 = _cuts(T)
    for scores in (np.random.default_rng(77).lognormal(0.0, 1.0, size=T).astype(np.float32),
                   np.random.default_rng(78).integers(0, 9, size=T).astype(np.float32),
                   wl.importance_scores(T, 1007)):
        st, bits = oracle.bits_from_scores(scores, n16, n8, n4)
        assert st == oracle.OK and np.array_equal(bits, by_library_sort(scores, n16, n8, n4))
    w = wl.WORKLOADS[4]
    assert wl.quantile_counts(w.n_tokens) == (410, 1228, 3277)
    from_oracle = wl.bits_for(w, rank_rule=lambda s, a, b, c: oracle.bits_from_scores(s, a, b, c)[1])
    assert np.array_equal(from_oracle, wl.bits_for(w, rank_rule=by_library_sort))


def test_bad_counts_are_rejected():
    st, _ = oracle.bits_from_scores(np.zeros(4, np.float32), 3, 2, 0)
    assert st == oracle.INVALID_ARG


# ----------------------------------------------------------------------------- combined score

def test_combined_score_special_cases():
    """Section 3.3's S = alpha I + (1 - alpha) T: alpha = 1 gives I, alpha = 0 gives T, equal inputs
    come back unchanged when alpha is a power of two, small integers combine exactly."""
    rng = np.random.default_rng(81)
    imp = rng.lognormal(0, 1, 500).astype(np.float32)
    tra = rng.lognormal(0, 1, 500).astype(np.float32)
    st, s1 = oracle.combine_scores(imp, tra, 1.0)
    assert st == oracle.OK and np.array_equal(s1, imp)
    st, s0 = oracle.combine_scores(imp, tra, 0.0)
    assert st == oracle.OK and np.array_equal(s0, tra)
    for alpha in (0.5, 0.25, 0.75):
        st, s = oracle.combine_scores(imp, imp, alpha)
        assert st == oracle.OK and np.array_equal(s, imp)
    a = rng.integers(0, 1000, 300).astype(np.float32)
    b = rng.integers(0, 1000, 300).astype(np.float32)
    st, s = oracle.combine_scores(a, b, 0.25)
    assert st == oracle.OK and np.array_equal(s.astype(np.float64), 0.25 * a.astype(np.float64) + 0.75 * b.astype(np.float64))
    for bad in (-0.1, 1.5, float("nan")):
        assert oracle.combine_scores(a, b, bad)[0] == oracle.INVALID_ARG


def test_combined_score_matches_numpy_float32_step_by_step():
    """The same three roundings with numpy's float32 scalars and arrays (each numpy operation
    rounds once); catches a fused multiply-add or double-precision intermediates in the C build."""
    rng = np.random.default_rng(82)
    imp = (rng.standard_normal(4000) * 3).astype(np.float32)
    tra = rng.lognormal(0, 2, 4000).astype(np.float32)
    for alpha in (0.3, 0.6180339887, 0.9):
        al = np.float32(alpha)
        want = al * imp + (np.float32(1.0) - al) * tra
        assert want.dtype == np.float32
        st, got = oracle.combine_scores(imp, tra, alpha)
        assert st == oracle.OK and np.array_equal(got.view(np.uint32), want.view(np.uint32))
        # and against the real-number expression: three roundings on the larger of the two terms
        # plus the rounding of 1 - alpha carried by T
        ta, tb = float(al) * imp.astype(np.float64), (1.0 - float(al)) * tra.astype(np.float64)
        big = np.maximum(np.maximum(np.abs(ta), np.abs(tb)), np.abs(ta + tb)).astype(np.float32)
        bound = 2 * np.spacing(big).astype(np.float64) + np.abs(tra).astype(np.float64) * 2.0 ** -24
        assert np.all(np.abs(got.astype(np.float64) - (ta + tb)) <= bound)
