"""Pins of the oracle's attention-from-the-card against what the definition fixes: special cases
with a known answer and the library routine it reduces to.  CPU only.

(The paper, Section 4.3, names consuming the quantised cache inside attention as the goal but
prints neither a formula nor numbers for it; the definition is the textbook one.)"""
import numpy as np
import pytest

import oracle
from paper_2605_03884_b200 import workloads as wl


def _card(Ks, Vs, bits, L, H, d, T, mode=0):
    lay = oracle.make_layout(L, H, d, T, bits_mode=mode)
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    return lay, card


def _cache(L, H, T, d, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    Ks = [(rng.standard_normal((H, T, d), dtype=np.float32) * scale).astype(np.float16) for _ in range(L)]
    Vs = [(rng.standard_normal((H, T, d), dtype=np.float32) * scale).astype(np.float16) for _ in range(L)]
    return Ks, Vs


def _reference_attention(Kh, Vh, q, per_kv, scale):
    """softmax(q K^T * scale) V with numpy in float64; Kh, Vh: per-layer [H, T, d]; q: [L, nq, d]."""
    L, nq, d = q.shape
    out = np.zeros((L, nq, d))
    for l in range(L):
        for j in range(nq):
            k = Kh[l][j // per_kv].astype(np.float64)
            v = Vh[l][j // per_kv].astype(np.float64)
            s = k @ q[l, j].astype(np.float64) * scale
            p = np.exp(s - s.max())
            out[l, j] = (p / p.sum()) @ v
    return out


def test_single_token_returns_its_value_row():
    L, H, d, T, nq = 2, 2, 64, 1, 4
    Ks, Vs = _cache(L, H, T, d, 1)
    lay, card = _card(Ks, Vs, np.full(T, 16, np.uint8), L, H, d, T)
    q = wl.random_fp16((L, nq, d), 2)
    st, o = oracle.card_attend(card, lay, q)
    assert st == oracle.OK
    for l in range(L):
        for j in range(nq):
            assert np.array_equal(o[l, j], Vs[l][j // 2][0].astype(np.float64))


def test_equal_value_rows_come_back_whatever_the_query():
    L, H, d, T, nq = 1, 2, 128, 37, 8
    Ks, Vs = _cache(L, H, T, d, 3)
    row = wl.random_fp16((H, 1, d), 4)
    Vs = [np.repeat(row, T, axis=1)]
    lay, card = _card(Ks, Vs, np.full(T, 16, np.uint8), L, H, d, T)
    st, o = oracle.card_attend(card, lay, wl.random_fp16((L, nq, d), 5, scale=3.0))
    assert st == oracle.OK
    for j in range(nq):
        np.testing.assert_allclose(o[0, j], row[j // 4, 0].astype(np.float64), rtol=1e-14, atol=1e-300)


def _rounding_bound(Kr, Vr, q, per_kv, scale):
    """How far attention over unrounded reconstructions can sit from attention over their FP16
    roundings (relative error 2^-11 per element): logits move by at most
    e = 2^-11 * scale * max_t sum_c |q_c K_tc|, weights by a factor within exp(+-2e), and the
    values themselves by 2^-11 relative."""
    L, nq, d = q.shape
    out = np.zeros((L, nq))
    for l in range(L):
        for j in range(nq):
            k = np.abs(Kr[l][j // per_kv].astype(np.float64))
            vmax = np.abs(Vr[l][j // per_kv].astype(np.float64)).max()
            e = 2.0 ** -11 * abs(scale) * (k @ np.abs(q[l, j].astype(np.float64))).max()
            out[l, j] = (np.exp(2 * e) - 1.0) * 2 * vmax + 2.0 ** -11 * vmax
    return out


def test_zero_query_gives_the_mean_of_the_record_values():
    """With q = 0 every weight is 1/T.  The mean of what the records stand for is within half an
    FP16 unit (relative 2^-11) of the mean of the injected FP16 values."""
    L, H, d, T, nq = 1, 1, 64, 50, 2
    Ks, Vs = _cache(L, H, T, d, 6)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.3, 0.1), 7)
    lay, card = _card(Ks, Vs, bits, L, H, d, T)
    Kr, Vr = [np.zeros_like(Ks[0])], [np.zeros_like(Vs[0])]
    assert oracle.card_inject(card, lay, Kr, Vr) == oracle.OK
    st, o = oracle.card_attend(card, lay, np.zeros((L, nq, d), np.float16))
    assert st == oracle.OK
    v = Vr[0][0].astype(np.float64)
    assert np.all(np.abs(o[0, 0] - v.mean(axis=0)) <= 2.0 ** -11 * np.abs(v).mean(axis=0) + 1e-12)
    np.testing.assert_allclose(o[0, 1], o[0, 0], rtol=0, atol=0)


def test_one_quantised_token_returns_code_times_scale_plus_zero():
    """T = 1: the output is the record's value row.  Checked on the hand-worked 4-bit group
    (scale 0.5, zero -1.5, codes 0,0,1,2,2,2,3,4,...: reconstruction -1.5 + 0.5 q, exact in FP16 too)."""
    L, H, d, T, nq = 1, 1, 64, 1, 1
    x = np.concatenate([np.arange(31) * 0.25 - 1.5, [6.0]]).astype(np.float16)
    V = np.concatenate([x, x]).reshape(1, 1, d)
    lay, card = _card([V.copy()], [V], np.full(T, 4, np.uint8), L, H, d, T)
    st, o = oracle.card_attend(card, lay, wl.random_fp16((L, nq, d), 3))
    assert st == oracle.OK
    codes = np.array([0, 0, 1, 2, 2, 2, 3, 4, 4, 4, 5, 6, 6, 6, 7, 8, 8, 8, 9, 10, 10, 10, 11, 12, 12, 12, 13, 14, 14, 14, 15, 15])
    want = -1.5 + 0.5 * np.concatenate([codes, codes])
    assert np.array_equal(o[0, 0], want)


def test_fp16_card_reduces_to_library_attention_on_the_original_cache():
    L, H, d, T, nq = 2, 2, 128, 200, 8
    Ks, Vs = _cache(L, H, T, d, 8)
    lay, card = _card(Ks, Vs, np.full(T, 16, np.uint8), L, H, d, T)
    q = wl.random_fp16((L, nq, d), 9)
    st, o = oracle.card_attend(card, lay, q)
    assert st == oracle.OK
    want = _reference_attention(Ks, Vs, q, nq // H, 1.0 / np.sqrt(d))
    np.testing.assert_allclose(o, want, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("mode", [0, 1])
def test_quantised_card_is_within_fp16_rounding_of_library_attention_on_the_injected_cache(mode):
    L, H, d, T, nq = 2, 3, 64, 150, 6
    Ks, Vs = _cache(L, H, T, d, 10)
    if mode == 0:
        bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 11)
    else:
        bits = np.concatenate([wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 20 + s) for s in range(L * H)])
    lay, card = _card(Ks, Vs, bits, L, H, d, T, mode)
    Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, lay, Kr, Vr) == oracle.OK
    q = wl.random_fp16((L, nq, d), 12)
    st, o = oracle.card_attend(card, lay, q, softmax_scale=0.3)
    assert st == oracle.OK
    ref = _reference_attention(Kr, Vr, q, nq // H, 0.3)
    bound = _rounding_bound(Kr, Vr, q, nq // H, 0.3)
    assert np.all(np.abs(o - ref).max(axis=2) <= bound)
    assert np.abs(o - ref).max() > 0          # and it is not the rounded cache that is attended to


@pytest.mark.parametrize("mode", [0, 1])
def test_injected_reading_is_library_attention_on_the_injected_cache(mode):
    """The second reading -- inject, then attend -- equals numpy softmax attention over exactly
    the FP16 arrays orc_card_inject writes, to double-precision rounding."""
    L, H, d, T, nq = 2, 3, 64, 150, 6
    Ks, Vs = _cache(L, H, T, d, 10)
    if mode == 0:
        bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 11)
    else:
        bits = np.concatenate([wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 20 + s) for s in range(L * H)])
    lay, card = _card(Ks, Vs, bits, L, H, d, T, mode)
    Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, lay, Kr, Vr) == oracle.OK
    q = wl.random_fp16((L, nq, d), 12)
    for scale in (0.3, 1.0 / np.sqrt(d), 2.0):
        st, o = oracle.card_attend(card, lay, q, softmax_scale=scale, injected=True)
        assert st == oracle.OK
        np.testing.assert_allclose(o, _reference_attention(Kr, Vr, q, nq // H, scale), rtol=1e-12, atol=1e-14)


def test_the_two_readings_coincide_on_fp16_tokens_and_differ_on_quantised_ones():
    L, H, d, T, nq = 1, 2, 128, 90, 4
    Ks, Vs = _cache(L, H, T, d, 15)
    q = wl.random_fp16((L, nq, d), 16)
    lay, card = _card(Ks, Vs, np.full(T, 16, np.uint8), L, H, d, T)
    a = oracle.card_attend(card, lay, q)[1]
    b = oracle.card_attend(card, lay, q, injected=True)[1]
    assert np.array_equal(a, b)
    lay, card = _card(Ks, Vs, np.full(T, 4, np.uint8), L, H, d, T)
    a = oracle.card_attend(card, lay, q)[1]
    b = oracle.card_attend(card, lay, q, injected=True)[1]
    Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, lay, Kr, Vr) == oracle.OK
    gap = np.abs(a - b).max(axis=2)
    assert gap.max() > 0 and np.all(gap <= _rounding_bound(Kr, Vr, q, nq // H, 1.0 / np.sqrt(d)))


def test_one_dominant_key_selects_its_value_row():
    """K rows are +-e_0 * 8 except token 17 = +e_0 * 64: with q = 32 e_0 the softmax weight of
    every other token is below exp(-64*32*... ) ~ 0, so the output is V[17] to double precision."""
    L, H, d, T, nq = 1, 1, 64, 40, 1
    K = np.zeros((H, T, d), np.float16)
    K[0, :, 0] = 8.0
    K[0, 17, 0] = 64.0
    V = wl.random_fp16((H, T, d), 13)
    lay, card = _card([K], [V], np.full(T, 16, np.uint8), L, H, d, T)
    q = np.zeros((L, nq, d), np.float16)
    q[0, 0, 0] = 32.0
    st, o = oracle.card_attend(card, lay, q, softmax_scale=1.0)
    assert st == oracle.OK
    np.testing.assert_allclose(o[0, 0], V[0, 17].astype(np.float64), rtol=1e-12, atol=1e-300)


def test_argument_and_card_checks():
    L, H, d, T = 1, 2, 64, 8
    Ks, Vs = _cache(L, H, T, d, 14)
    lay, card = _card(Ks, Vs, np.full(T, 4, np.uint8), L, H, d, T)
    st, _ = oracle.card_attend(card, lay, np.zeros((L, 3, d), np.float16))     # 3 query heads over 2 KV heads
    assert st == oracle.INVALID_ARG
    bad = card.copy()
    bad[0] ^= 0xFF
    st, _ = oracle.card_attend(bad, lay, np.zeros((L, 2, d), np.float16))
    assert st == oracle.BAD_CARD
