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
