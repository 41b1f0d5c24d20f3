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


# ----------------------------------------------------------------------------- byte budget

def _rec(d, meta=8):
    return [oracle.record_bytes(d, b, meta) for b in (2, 4, 8, 16)]


def _stream_bytes(bits, d, meta=8):
    r = dict(zip((2, 4, 8, 16), _rec(d, meta)))
    return sum(r[int(b)] for b in bits)


def test_budget_rule_special_cases_with_known_answers():
    """Budget for 2 bits only -> all 2; for FP16 everywhere -> all 16; equal scores and exactly the
    bytes of 4 bits everywhere -> all 4 (a lower rung always comes first among equal scores); one
    token so far above the rest that its third upgrade outweighs anybody's first -> it alone climbs."""
    d, T = 128, 50
    r2, r4, r8, r16 = _rec(d)
    s = np.random.default_rng(1).lognormal(0, 1, T).astype(np.float32)
    st, bits = oracle.bits_from_scores_budget(s, d, T * r2)
    assert st == oracle.OK and np.all(bits == 2)
    st, bits = oracle.bits_from_scores_budget(s, d, T * r16)
    assert st == oracle.OK and np.all(bits == 16)
    st, bits = oracle.bits_from_scores_budget(s, d, T * r16 + 12345)
    assert st == oracle.OK and np.all(bits == 16)
    st, bits = oracle.bits_from_scores_budget(np.ones(T, np.float32), d, T * r4)
    assert st == oracle.OK and np.all(bits == 4)
    st, bits = oracle.bits_from_scores_budget(np.ones(T, np.float32), d, T * r4 + 3 * (r8 - r4) + 5)
    assert st == oracle.OK and bits.tolist() == [8] * 3 + [4] * (T - 3)           # equal keys: lower index first
    s = np.ones(T, np.float32)
    s[17] = 2.0 ** 20                                                             # 2^20 * 2^-23 > 1 * 2^-9 ?  no: 2^-3 > 2^-9, yes
    st, bits = oracle.bits_from_scores_budget(s, d, T * r2 + (r16 - r2))
    assert st == oracle.OK and bits[17] == 16 and np.all(np.delete(bits, 17) == 2)
    assert oracle.bits_from_scores_budget(s, d, T * r2 - 1)[0] == oracle.BUFFER_TOO_SMALL
    bad = s.copy()
    bad[3] = -1.0
    assert oracle.bits_from_scores_budget(bad, d, T * r16)[0] == oracle.INVALID_ARG
    assert oracle.bits_from_scores_budget(s, d, T * r16, weights=(1.0, 2.0, 0.5))[0] == oracle.INVALID_ARG


@pytest.mark.parametrize("d,meta", [(128, 8), (64, 8), (128, 4)])
def test_budget_is_respected_and_the_next_upgrade_would_not_fit(d, meta):
    """Over a sweep of budgets: the stream never exceeds the budget; with power-of-two weights the
    keys are exact, so more important tokens never get fewer bits; and what is left of the budget
    is less than the cost of the upgrade that comes next in the order (recomputed here with
    Python's sort on (-key, rung, index))."""
    T = 200
    rec = _rec(d, meta)
    s = np.random.default_rng(2).lognormal(0, 1.5, T).astype(np.float32)
    w = oracle.DEFAULT_UPGRADE_WEIGHTS
    order = sorted(((-(np.float32(s[t]) * np.float32(w[i])), i, t) for t in range(T) for i in range(3)))
    for budget in range(T * rec[0], T * rec[3] + 1, 997):
        st, bits = oracle.bits_from_scores_budget(s, d, budget, meta_bytes=meta)
        assert st == oracle.OK
        used = _stream_bytes(bits, d, meta)
        assert used <= budget
        by_score = np.argsort(-s, kind="stable")
        assert np.all(np.diff(bits[by_score].astype(int)) <= 0)
        level = {2: 0, 4: 1, 8: 2, 16: 3}
        granted = sum(level[int(b)] for b in bits)
        if granted < 3 * T:
            _, rung, t = order[granted]
            assert level[int(bits[t])] == rung                       # the next upgrade in the order is this token's next rung
            assert rec[rung + 1] - rec[rung] > budget - used         # and it does not fit
        for j in range(granted):                                     # everything before it was granted
            _, rung, t = order[j]
            assert level[int(bits[t])] > rung


def test_budget_rule_is_the_best_use_of_the_bytes_it_spends():
    """Brute force on tiny inputs: among ALL assignments of {2,4,8,16} to T tokens that cost no more
    than what the rule spent, none removes more weighted error (sum of key * cost over granted
    upgrades) -- the rule takes upgrades in order of worth per byte, so at its own spending it is the
    optimum of the knapsack in Section 3.3's objective under the additive error model."""
    import itertools
    d, T = 128, 6
    rec = _rec(d)
    cost = [rec[i + 1] - rec[i] for i in range(3)]
    w = [float(np.float32(x)) for x in oracle.DEFAULT_UPGRADE_WEIGHTS]
    rng = np.random.default_rng(3)
    for trial in range(4):
        s = rng.lognormal(0, 2.0, T).astype(np.float32)
        for budget in (T * rec[0] + 100, T * rec[0] + 700, T * rec[1] + 333, T * rec[2] + 50):
            st, bits = oracle.bits_from_scores_budget(s, d, budget)
            assert st == oracle.OK
            level = [{2: 0, 4: 1, 8: 2, 16: 3}[int(b)] for b in bits]
            spent = sum(sum(cost[:l]) for l in level)
            worth = sum(float(s[t]) * w[i] * cost[i] for t in range(T) for i in range(level[t]))
            best = 0.0
            for assign in itertools.product(range(4), repeat=T):
                c = sum(sum(cost[:l]) for l in assign)
                if c <= spent:
                    best = max(best, sum(float(s[t]) * w[i] * cost[i] for t in range(T) for i in range(assign[t])))
            assert worth >= best * (1 - 1e-12)


def test_budget_rule_is_a_rank_rule_with_the_counts_it_arrives_at():
    """Distinct scores and power-of-two weights: the outcome equals the rank rule run with the
    class counts the budget rule produced (ties the two functions to each other)."""
    d, T = 128, 3000
    rec = _rec(d)
    s = np.unique(np.random.default_rng(4).lognormal(0, 1, 2 * T).astype(np.float32))[:T].copy()
    np.random.default_rng(5).shuffle(s)
    for budget in (T * rec[0] + 5000, T * 80, T * 120, T * 200):
        st, bits = oracle.bits_from_scores_budget(s, d, budget)
        assert st == oracle.OK
        n16, n8, n4 = int((bits == 16).sum()), int((bits == 8).sum()), int((bits == 4).sum())
        st, ranked = oracle.bits_from_scores(s, n16, n8, n4)
        assert st == oracle.OK and np.array_equal(bits, ranked)
        assert np.array_equal(bits, by_library_sort(s, n16, n8, n4))


# ---------------------------------------------------------------------------------------------
# The controller of Section 4.1.2 (two-layer perceptron over six features -> one of four widths)

def _pack(w1, b1, w2, b2):
    return np.concatenate([np.asarray(w1, np.float32).reshape(-1), np.asarray(b1, np.float32).reshape(-1),
                           np.asarray(w2, np.float32).reshape(-1), np.asarray(b2, np.float32).reshape(-1)])


def test_controller_with_hand_set_weights_follows_the_rule_it_encodes():
    """hidden_0 = relu(x0 - 1), hidden_1 = relu(x0 - 2), hidden_2 = relu(x0 - 3); outputs
    (0.5, h0, 2 h1, 4 h2): the winner changes at x0 = 1.5, 2.5, 3.5 -- worked out by hand."""
    w1 = np.zeros((3, 6)); w1[:, 0] = 1.0
    b1 = [-1.0, -2.0, -3.0]
    w2 = np.zeros((4, 3)); w2[1, 0] = 1.0; w2[2, 1] = 2.0; w2[3, 2] = 4.0
    b2 = [0.5, 0.0, 0.0, 0.0]
    x = np.zeros((8, 6), np.float32)
    x[:, 0] = [0.0, 1.25, 1.75, 2.25, 2.75, 3.25, 3.75, 10.0]
    x[:, 1:] = 7.0   # features the network does not look at
    st, bits, outs = oracle.bits_from_features(x, 3, _pack(w1, b1, w2, b2))
    assert st == oracle.OK
    # x0: outputs -> winner
    #  0.00: (0.5, 0,    0,   0)  -> 2      1.25: (0.5, 0.25, 0,   0)  -> 2
    #  1.75: (0.5, 0.75, 0,   0)  -> 4      2.25: (0.5, 1.25, 0.5, 0)  -> 4
    #  2.75: (0.5, 1.75, 1.5, 0)  -> 4      3.25: (0.5, 2.25, 2.5, 1)  -> 8
    #  3.75: (0.5, 2.75, 3.5, 3)  -> 8     10.00: (0.5, 9,    16,  28) -> 16
    assert bits.tolist() == [2, 2, 4, 4, 4, 8, 8, 16]
    assert outs[5].tolist() == [0.5, 2.25, 2.5, 1.0] and outs[7].tolist() == [0.5, 9.0, 16.0, 28.0]


def test_controller_rectifies_the_hidden_layer():
    """One hidden unit with a negative pre-activation and a negative outgoing weight: without the
    rectifier class 1 would win (-1 * -3 = 3); with it the unit is silent and the bias decides."""
    w1 = np.zeros((1, 6)); w1[0, 2] = 1.0
    w2 = np.zeros((4, 1)); w2[1, 0] = -1.0
    x = np.zeros((2, 6), np.float32); x[0, 2] = -3.0; x[1, 2] = 3.0
    st, bits, outs = oracle.bits_from_features(x, 1, _pack(w1, [0.0], w2, [0.0, 0.0, 1.0, 0.0]))
    assert st == oracle.OK and bits.tolist() == [8, 8]
    assert outs[0].tolist() == [0.0, 0.0, 1.0, 0.0] and outs[1].tolist() == [0.0, -3.0, 1.0, 0.0]


def test_controller_ties_go_to_fewer_bits_and_biases_alone_decide_without_weights():
    x = np.random.default_rng(3).standard_normal((5, 6)).astype(np.float32)
    for b2, want in (([1, 1, 1, 1], 2), ([0, 2, 2, 1], 4), ([0, 0, 3, 3], 8), ([0, 0, 0, 1], 16)):
        st, bits, _ = oracle.bits_from_features(x, 4, _pack(np.zeros((4, 6)), np.zeros(4), np.zeros((4, 4)), b2))
        assert st == oracle.OK and np.all(bits == want)


def test_controller_against_numpy_float32_step_by_step():
    """The same network with numpy float32 scalars, one rounded operation at a time in the stated
    order (bias first, then the terms by index)."""
    rng = np.random.default_rng(11)
    hidden = 46   # 11 * 46 + 4 = 510 parameters: the size nearest to the paper's 512 for this shape
    w1 = rng.standard_normal((hidden, 6)).astype(np.float32)
    b1 = rng.standard_normal(hidden).astype(np.float32)
    w2 = rng.standard_normal((4, hidden)).astype(np.float32)
    b2 = rng.standard_normal(4).astype(np.float32)
    x = rng.standard_normal((300, 6)).astype(np.float32)
    st, bits, outs = oracle.bits_from_features(x, hidden, _pack(w1, b1, w2, b2))
    assert st == oracle.OK
    ladder = [2, 4, 8, 16]
    for t in range(x.shape[0]):
        hid = []
        for j in range(hidden):
            acc = np.float32(b1[j])
            for i in range(6):
                acc = np.float32(acc + np.float32(w1[j, i] * x[t, i]))
            hid.append(acc if acc > 0 else np.float32(0.0))
        out = []
        for k in range(4):
            acc = np.float32(b2[k])
            for j in range(hidden):
                acc = np.float32(acc + np.float32(w2[k, j] * hid[j]))
            out.append(acc)
        assert [float(o) for o in out] == outs[t].tolist()
        assert bits[t] == ladder[int(np.argmax(out))]   # numpy's argmax also takes the first of equals
    assert len(set(bits.tolist())) == 4                 # every width occurs


def test_controller_outputs_are_close_to_the_matrix_form():
    """Against the library routine: relu(x W1^T + b1) W2^T + b2 in float64 -- equal up to the
    rounding of float32 sums, and the same widths wherever the two largest outputs are not close."""
    rng = np.random.default_rng(12)
    hidden = 46
    w1, b1 = rng.standard_normal((hidden, 6)), rng.standard_normal(hidden)
    w2, b2 = rng.standard_normal((4, hidden)), rng.standard_normal(4)
    x = rng.standard_normal((2000, 6))
    st, bits, outs = oracle.bits_from_features(x, hidden, _pack(w1, b1, w2, b2))
    f32 = lambda a: np.asarray(a, np.float32).astype(np.float64)
    ref = np.maximum(f32(x) @ f32(w1).T + f32(b1), 0.0) @ f32(w2).T + f32(b2)
    assert np.abs(outs - ref).max() < 1e-4
    top2 = np.sort(ref, axis=1)[:, -2:]
    clear = top2[:, 1] - top2[:, 0] > 1e-3
    assert clear.sum() > 1900
    assert np.array_equal(bits[clear], np.array([2, 4, 8, 16])[np.argmax(ref, axis=1)][clear])


def test_controller_argument_checks():
    x = np.zeros((1, 6), np.float32)
    for hidden in (0, 129):
        import ctypes as C
        bits = np.zeros(1, np.uint8)
        p = np.zeros(11 * 129 + 4, np.float32)
        st = oracle.lib().orc_bits_from_features(x.ctypes.data_as(C.c_void_p), 1, hidden, p.ctypes.data_as(C.c_void_p),
                                                 bits.ctypes.data_as(C.c_void_p), None)
        assert st == oracle.INVALID_ARG
