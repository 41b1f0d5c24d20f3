"""Rank-based bit-width assignment on the GPU against the oracle (exact), through the C-ABI."""
import numpy as np
import pytest

import oracle
import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from paper_2605_03884_b200 import workloads as wl
from gpu_utils import gpu_create, padded_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _library():
    qbuild.build()
    q.load_library()


def _gpu_bits(scores, n16, n8, n4):
    import torch
    sd = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).cuda()
    bd = torch.full(scores.shape, 0xEE, dtype=torch.uint8, device="cuda")
    q.bits_from_scores(sd, n16, n8, n4, bd)
    torch.cuda.synchronize()
    return bd.cpu().numpy()


def _cuts(T):
    c16 = int(np.floor(0.05 * T + 0.5)); c8 = int(np.floor(0.20 * T + 0.5)); c4 = int(np.floor(0.60 * T + 0.5))
    return c16, c8 - c16, c4 - c8


@pytest.mark.parametrize("T", [1, 3, 63, 64, 65, 1023, 1024, 1025, 8192, 20000])
def test_random_scores(T):
    scores = np.random.default_rng(T).lognormal(0.0, 1.0, size=T).astype(np.float32)
    n16, n8, n4 = _cuts(T)
    st, want = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == oracle.OK
    assert np.array_equal(_gpu_bits(scores, n16, n8, n4), want)


@pytest.mark.parametrize("levels", [1, 2, 5])
def test_ties_go_to_the_lower_index(levels):
    T = 3000
    scores = np.random.default_rng(levels).integers(0, levels, size=T).astype(np.float32)
    st, want = oracle.bits_from_scores(scores, 123, 456, 789)
    assert st == oracle.OK
    assert np.array_equal(_gpu_bits(scores, 123, 456, 789), want)


def test_extreme_splits_and_special_values():
    T = 500
    scores = np.random.default_rng(9).standard_normal(T).astype(np.float32)
    scores[::7] = -0.0
    scores[1::7] = 0.0            # equal to -0.0
    scores[3] = np.float32(3e38)
    scores[4] = np.float32(-3e38)
    scores[5] = np.float32(1e-45)  # subnormal
    for split in ((0, 0, 0), (T, 0, 0), (0, T, 0), (0, 0, T), (1, 1, 1), (100, 0, 400)):
        st, want = oracle.bits_from_scores(scores, *split)
        assert st == oracle.OK
        assert np.array_equal(_gpu_bits(scores, *split), want)


def test_segments_are_ranked_independently():
    S, T = 6, 777
    scores = np.random.default_rng(11).standard_normal((S, T)).astype(np.float32)
    got = _gpu_bits(scores, 40, 120, 300)
    for s in range(S):
        st, want = oracle.bits_from_scores(scores[s], 40, 120, 300)
        assert st == oracle.OK and np.array_equal(got[s], want)


def test_argument_checks():
    import torch
    sd = torch.zeros(16, dtype=torch.float32, device="cuda")
    bd = torch.zeros(16, dtype=torch.uint8, device="cuda")
    assert q.bits_from_scores(sd, 10, 5, 2, bd, check=False) == q.binding.ERR_INVALID_ARG
    assert q.bits_from_scores(sd, -1, 0, 0, bd, check=False) == q.binding.ERR_INVALID_ARG


def test_scores_to_card_end_to_end():
    """Scores -> bit-widths on the GPU -> card on the GPU equals the oracle's card from the oracle's bit-widths."""
    import torch
    L, H, d, T = 2, 2, 128, 1500
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=71)
    scores = np.random.default_rng(72).lognormal(0.0, 1.0, size=T).astype(np.float32)
    n16, n8, n4 = _cuts(T)
    st, bits_o = oracle.bits_from_scores(scores, n16, n8, n4)
    st_o, want = oracle.card_create(oracle.make_layout(L, H, d, T), Ks, Vs, bits_o)
    assert st == oracle.OK and st_o == oracle.OK
    bits_g = _gpu_bits(scores, n16, n8, n4)
    st_g, hdr, whole, cap = gpu_create(q, q.make_layout(L, H, d, T), Ks, Vs, bits_g)
    assert st_g == 0 and np.array_equal(whole[:want.size], want)


def test_combined_score_bit_exact_and_feeds_the_rank_rule():
    import torch
    rng = np.random.default_rng(83)
    n = 8192 + 37
    imp = rng.lognormal(0, 1, n).astype(np.float32)
    tra = (rng.standard_normal(n) * 2).astype(np.float32)
    for alpha in (0.0, 0.3, 0.6180339887, 1.0):
        st, want = oracle.combine_scores(imp, tra, alpha)
        assert st == oracle.OK
        out = torch.full((n,), -7.0, dtype=torch.float32, device="cuda")
        q.combine_scores(torch.from_numpy(imp).cuda(), torch.from_numpy(tra).cuda(), alpha, out)
        got = out.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # in place, then straight into the rank rule
    st, want = oracle.combine_scores(imp, tra, 0.4)
    stb, bits_want = oracle.bits_from_scores(want, 400, 1200, 3300)
    buf = torch.from_numpy(imp).cuda()
    q.combine_scores(buf, torch.from_numpy(tra).cuda(), 0.4, buf)
    bits = torch.zeros(n, dtype=torch.uint8, device="cuda")
    q.bits_from_scores(buf, 400, 1200, 3300, bits)
    assert stb == oracle.OK and np.array_equal(bits.cpu().numpy(), bits_want)
    with pytest.raises(q.QkvsError) as e:
        q.combine_scores(buf, buf, 1.5, buf)
    assert e.value.status == q.binding.ERR_INVALID_ARG


# ----------------------------------------------------------------------------- larger inputs, byte budget

@pytest.mark.parametrize("T", [131072, 1 << 20])
def test_rank_rule_at_long_contexts(T):
    """Up to the limit of 2^20 tokens, with a block of equal scores across the cuts."""
    scores = np.random.default_rng(T).lognormal(0.0, 1.0, size=T).astype(np.float32)
    scores[T // 3: T // 3 + T // 4] = np.float32(1.0)
    n16, n8, n4 = _cuts(T)
    st, want = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == oracle.OK
    assert np.array_equal(_gpu_bits(scores, n16, n8, n4), want)


def _gpu_budget(scores, d, budget, weights=None, meta=8, with_offsets=True):
    import torch
    sd = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).cuda()
    bd = torch.full(scores.shape, 0xEE, dtype=torch.uint8, device="cuda")
    shape = (scores.shape[0], scores.shape[1] + 1) if scores.ndim == 2 else (scores.shape[0] + 1,)
    od = torch.full(shape, -1, dtype=torch.int32, device="cuda") if with_offsets else None
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    q.bits_from_scores_budget(sd, d, budget, bd, weights=weights, meta_bytes=meta, offsets_dev=od, status_dev=status)
    torch.cuda.synchronize()
    return bd.cpu().numpy(), (od.cpu().numpy().view(np.uint32) if with_offsets else None), int(status.item())


@pytest.mark.parametrize("T", [1, 2, 7, 64, 1000, 8192, 20000, 131072, 1 << 20])
def test_budget_rule_random_scores(T):
    d = 128
    r2, r16 = oracle.record_bytes(d, 2), oracle.record_bytes(d, 16)
    scores = np.random.default_rng(100 + T).lognormal(0.0, 1.5, size=T).astype(np.float32)
    budgets = [T * r2, T * r2 + 31, T * 80, T * 100 + 17, T * 150, T * r16 - 1, T * r16, T * r16 + 999]
    for budget in budgets if T <= 20000 else budgets[2:5]:
        st, want = oracle.bits_from_scores_budget(scores, d, budget)
        assert st == oracle.OK
        got, off, status = _gpu_budget(scores, d, budget)
        assert status == 0 and np.array_equal(got, want), (T, budget)
        st, off_want, _ = oracle.scan_offsets(d, want)
        assert st == oracle.OK and np.array_equal(off, off_want)
        assert int(off[-1]) <= budget


@pytest.mark.parametrize("levels", [1, 2, 5])
def test_budget_rule_with_many_equal_scores(levels):
    """Few distinct scores: the budget runs out in the middle of a block of equal keys, which is
    then granted by rung and by index."""
    d, T = 128, 5000
    scores = np.random.default_rng(levels).integers(0, levels, size=T).astype(np.float32)
    for budget in (T * 64 + 32 * 77, T * 96 + 64 * 1234 + 7, T * 160 + 96 * 4999, T * 70):
        for weights in (None, (1.0, 1.0, 1.0), (0.3, 0.07, 0.07)):
            st, want = oracle.bits_from_scores_budget(scores, d, budget, **({} if weights is None else {"weights": weights}))
            assert st == oracle.OK
            got, _, status = _gpu_budget(scores, d, budget, weights)
            assert status == 0 and np.array_equal(got, want), (levels, budget, weights)


@pytest.mark.parametrize("d,meta", [(64, 8), (128, 4), (256, 8), (192, 8)])
def test_budget_rule_other_record_sizes(d, meta):
    T = 3000
    scores = np.random.default_rng(d + meta).lognormal(0.0, 1.0, size=T).astype(np.float32)
    scores[::11] = 0.0
    scores[1::11] = -0.0
    r2 = oracle.record_bytes(d, 2, meta)
    for budget in (T * r2 + 100, T * r2 * 2, T * r2 * 3 + 5):
        st, want = oracle.bits_from_scores_budget(scores, d, budget, meta_bytes=meta)
        assert st == oracle.OK
        got, off, status = _gpu_budget(scores, d, budget, meta=meta)
        assert status == 0 and np.array_equal(got, want)
        assert np.array_equal(off, oracle.scan_offsets(d, want, meta)[1])


def test_budget_rule_segments_bad_scores_and_arguments():
    import torch
    d, S, T = 128, 5, 900
    scores = np.random.default_rng(21).lognormal(0.0, 1.0, size=(S, T)).astype(np.float32)
    got, off, status = _gpu_budget(scores, d, T * 100)
    assert status == 0
    for s in range(S):
        st, want = oracle.bits_from_scores_budget(scores[s], d, T * 100)
        assert st == oracle.OK and np.array_equal(got[s], want)
        assert np.array_equal(off[s], oracle.scan_offsets(d, want)[1])
    bad = scores.copy()
    bad[2, 17] = -0.5
    bad[4, 3] = np.nan
    got, _, status = _gpu_budget(bad, d, T * 100, with_offsets=False)
    assert status == q.binding.ERR_INVALID_ARG and np.all(got[2] == 2) and np.all(got[4] == 2)
    assert np.array_equal(got[0], oracle.bits_from_scores_budget(scores[0], d, T * 100)[1])
    sd = torch.zeros(16, dtype=torch.float32, device="cuda")
    bd = torch.zeros(16, dtype=torch.uint8, device="cuda")
    assert q.bits_from_scores_budget(sd, 128, 16 * 64 - 1, bd, check=False) == q.binding.ERR_BUFFER_TOO_SMALL
    assert q.bits_from_scores_budget(sd, 96, 16 * 256, bd, check=False) == q.binding.ERR_UNSUPPORTED_SHAPE
    assert q.bits_from_scores_budget(sd, 128, 16 * 256, bd, weights=(1.0, 2.0, 1.0), check=False) == q.binding.ERR_INVALID_ARG


def test_budgeted_scores_to_card_end_to_end():
    """Scores -> bit-widths under a budget on the GPU -> card: the card's streams keep to the budget
    and the card equals the oracle's from the oracle's bit-widths."""
    L, H, d, T = 2, 2, 128, 1500
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=73)
    scores = np.random.default_rng(74).lognormal(0.0, 1.0, size=T).astype(np.float32)
    budget = T * 96                                    # the bytes of a uniform 4-bit stream
    st, bits_o = oracle.bits_from_scores_budget(scores, d, budget)
    st_o, want = oracle.card_create(oracle.make_layout(L, H, d, T), Ks, Vs, bits_o)
    assert st == oracle.OK and st_o == oracle.OK
    bits_g, off, status = _gpu_budget(scores, d, budget)
    st_g, hdr, whole, cap = gpu_create(q, q.make_layout(L, H, d, T), Ks, Vs, bits_g)
    assert st_g == 0 and np.array_equal(whole[:want.size], want)
    assert hdr.stream_bytes <= budget and hdr.stream_bytes == int(off[-1])


def _controller_params(rng, hidden):
    return np.concatenate([rng.standard_normal(6 * hidden), rng.standard_normal(hidden),
                           rng.standard_normal(4 * hidden), rng.standard_normal(4)]).astype(np.float32)


@pytest.mark.parametrize("n,hidden", [(1, 1), (37, 46), (8192, 46), (100003, 46), (5000, 128)])
def test_controller_bit_exact(n, hidden):
    """The two-layer controller: outputs equal bit for bit, hence the same bit-widths."""
    import torch
    rng = np.random.default_rng(1000 + n + hidden)
    x = rng.standard_normal((n, 6)).astype(np.float32)
    params = _controller_params(rng, hidden)
    st, want_bits, want_out = oracle.bits_from_features(x, hidden, params)
    assert st == oracle.OK
    bits = torch.full((n,), 99, dtype=torch.uint8, device="cuda")
    outs = torch.full((n, 4), -7.0, dtype=torch.float32, device="cuda")
    q.bits_from_features(torch.from_numpy(x).cuda(), hidden, torch.from_numpy(params).cuda(), bits, outs)
    assert np.array_equal(outs.cpu().numpy().view(np.uint32), want_out.view(np.uint32))
    assert np.array_equal(bits.cpu().numpy(), want_bits)
    # without the optional outputs
    bits2 = torch.full((n,), 99, dtype=torch.uint8, device="cuda")
    q.bits_from_features(torch.from_numpy(x).cuda(), hidden, torch.from_numpy(params).cuda(), bits2)
    assert np.array_equal(bits2.cpu().numpy(), want_bits)


def test_controller_ties_special_values_and_a_card_from_its_bits():
    import torch
    from gpu_utils import gpu_create, padded_cache
    rng = np.random.default_rng(77)
    hidden = 8
    # all weights zero: the biases decide, equal ones go to the fewer bits
    for b2, want in (([1, 1, 1, 1], 2), ([0, 2, 2, 1], 4), ([0, 0, 0, 1], 16)):
        params = np.concatenate([np.zeros(11 * hidden), np.asarray(b2, np.float64)]).astype(np.float32)
        bits = torch.zeros(50, dtype=torch.uint8, device="cuda")
        q.bits_from_features(torch.from_numpy(rng.standard_normal((50, 6)).astype(np.float32)).cuda(), hidden,
                             torch.from_numpy(params).cuda(), bits)
        assert bool((bits == want).all())
    # infinities and a not-a-number among the features: whatever comes out, both sides agree
    x = rng.standard_normal((64, 6)).astype(np.float32)
    x[3, 0] = np.inf
    x[4, 1] = -np.inf
    x[5, 2] = np.nan
    params = _controller_params(rng, hidden)
    st, want_bits, _ = oracle.bits_from_features(x, hidden, params)
    bits = torch.zeros(64, dtype=torch.uint8, device="cuda")
    q.bits_from_features(torch.from_numpy(x).cuda(), hidden, torch.from_numpy(params).cuda(), bits)
    assert st == oracle.OK and np.array_equal(bits.cpu().numpy(), want_bits)
    # features -> bits -> card, all on the device, against the oracle's card from the oracle's bits
    L, H, d, T = 1, 2, 128, 333
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=78)
    feats = rng.standard_normal((T, 6)).astype(np.float32)
    st, obits, _ = oracle.bits_from_features(feats, hidden, params)
    _, want = oracle.card_create(oracle.make_layout(L, H, d, T), Ks, Vs, obits)
    gbits = torch.zeros(T, dtype=torch.uint8, device="cuda")
    q.bits_from_features(torch.from_numpy(feats).cuda(), hidden, torch.from_numpy(params).cuda(), gbits)
    st, hdr, whole, _ = gpu_create(q, q.make_layout(L, H, d, T), Ks, Vs, gbits.cpu().numpy())
    assert st == q.binding.OK and np.array_equal(whole[:want.size], want)
