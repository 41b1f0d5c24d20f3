"""Pins of the oracle's wider-group variant (groups of 64 or 128 channels, Section 3.1: the fewer
pairs of scale and zero a record carries, the closer it comes to 0.5 bytes per element at 4 bits).
CPU only.  What is pinned: record and card sizes against the closed form written out here; the
quantiser against step-by-step IEEE arithmetic in rationals; the special case in which a wide
group's halves span the same range as the whole, where it must give the codes of the groups of
32 (pinned on their own); the error bound; packing and record layout against numpy; whole cards
through injection and attention against the same statements made with groups of 32."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_03884_b200 import workloads as wl
from test_oracle_pins import _frac16, _rn32


def _pairs_bytes(d, meta, group):
    raw = meta * (d // group)
    return raw if group == 32 else (raw + 15) // 16 * 16


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("group", [32, 64, 128])
@pytest.mark.parametrize("meta", [8, 4])
def test_record_sizes_follow_the_closed_form(d, group, meta):
    for b in (2, 4, 8):
        assert oracle.record_bytes(d, b, meta, group) == d * b // 8 + _pairs_bytes(d, meta, group)
        assert oracle.record_bytes(d, b, meta, group) % 16 == 0
    assert oracle.record_bytes(d, 16, meta, group) == 2 * d
    assert oracle.record_bytes(d, 3, meta, group) == -1
    assert oracle.record_bytes(d, 4, meta, 48) == -1


def test_effective_bits_at_four_bits():
    """Bytes per element at 4 bits: 0.75 with fp32 pairs per 32 channels; 0.5625 at head_dim 256
    with one FP16 pair per 128 channels (padded to 16 bytes) -- the padding is what keeps
    head_dim 128 at 0.625 whatever the group."""
    assert oracle.record_bytes(128, 4, 8, 32) / 128 == 0.75
    assert oracle.record_bytes(128, 4, 4, 32) / 128 == 0.625
    assert oracle.record_bytes(128, 4, 8, 64) / 128 == 0.625
    assert oracle.record_bytes(128, 4, 4, 128) / 128 == 0.625
    assert oracle.record_bytes(256, 4, 4, 128) / 256 == 0.5625
    assert oracle.record_bytes(256, 4, 8, 128) / 256 == 0.5625
    assert oracle.record_bytes(256, 4, 8, 64) / 256 == 0.625


@pytest.mark.parametrize("n", [64, 128])
@pytest.mark.parametrize("b", [2, 4, 8])
def test_step_by_step_ieee_emulation_in_rationals(n, b):
    qmax = (1 << b) - 1
    rng = np.random.default_rng(100 * n + b)
    for trial in range(12):
        x = (rng.standard_normal(n, dtype=np.float32) * np.float32([1.0, 30.0, 1e-3][trial % 3])).astype(np.float16)
        scale, zero, q = oracle.quantize_span(x, b)
        deq = oracle.dequantize_span(q, scale, zero)
        fx = [_frac16(v) for v in x]
        mn, mx = min(fx), max(fx)
        rng_ = _rn32(mx - mn)
        sc, inv = _rn32(rng_ / qmax), _rn32(Fraction(qmax) / rng_)
        assert Fraction(float(scale)) == sc and Fraction(float(zero)) == mn
        for i in range(n):
            u = _rn32(_rn32(fx[i] - mn) * inv)
            fl = u.numerator // u.denominator
            rem = u - fl
            code = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2) else 0)
            assert int(q[i]) == min(code, qmax)
            r = _rn32(_rn32(int(q[i]) * sc) + mn)
            assert float(deq[i]) == float(np.float32(float(r)).astype(np.float16))
            assert abs(fx[i] - Fraction(float(deq[i]))) <= sc / 2 + Fraction(1, 2048) * max(abs(mn), abs(mx)) + Fraction(1, 10 ** 6)


@pytest.mark.parametrize("n", [64, 128])
@pytest.mark.parametrize("compact", [False, True])
def test_halves_with_the_range_of_the_whole_give_the_codes_of_groups_of_32(n, compact):
    """Every 32 of the n values contain the same minimum and maximum: the wide group then has the
    scale and zero of each group of 32, hence their codes (hand-worked example A's values, with
    exact ties, in each 32)."""
    base = np.concatenate([np.arange(31) * 0.25 - 1.5, [6.0]]).astype(np.float16)
    rng = np.random.default_rng(n)
    x = np.concatenate([rng.permutation(base) for _ in range(n // 32)])
    for b in (2, 4, 8):
        scale, zero, q = oracle.quantize_span(x, b, compact=compact)
        for j in range(n // 32):
            part = x[32 * j:32 * j + 32]
            s32, z32, q32 = (oracle.quantize_group_compact(part, b) if compact else oracle.quantize_group(part, b))
            assert float(s32) == float(scale) and float(z32) == float(zero)
            assert np.array_equal(q32, q[32 * j:32 * j + 32])


def test_wider_groups_never_have_a_smaller_scale():
    """The range of a union is at least the range of each part: the price of fewer pairs."""
    rng = np.random.default_rng(7)
    x = rng.standard_normal(128, dtype=np.float32).astype(np.float16)
    x[5] = np.float16(9.0)       # an outlier channel, as keys have them
    s128 = float(oracle.quantize_span(x, 4)[0])
    s64 = [float(oracle.quantize_span(x[i:i + 64], 4)[0]) for i in (0, 64)]
    s32 = [float(oracle.quantize_group(x[i:i + 32], 4)[0]) for i in range(0, 128, 32)]
    assert s128 >= max(s64) and max(s64[0], s64[1]) >= max(s32)
    assert s64[0] >= max(s32[:2]) and s64[1] >= max(s32[2:])
    assert s128 == s64[0] > s64[1]                 # the outlier stretches every group it is in


@pytest.mark.parametrize("group,meta", [(64, 8), (128, 8), (64, 4), (128, 4)])
def test_record_layout_pairs_padding_codes(group, meta):
    """A record is: the pairs, zero bytes up to a multiple of 16, the little-endian code bit-string
    of the whole row (numpy packbits, group after group)."""
    d, T = 256, 5
    x = wl.random_fp16((T, d), 40 + group + meta)
    bits = np.array([4, 2, 8, 16, 4], np.uint8)
    payload = oracle.encode_stream(x, bits, meta, group)
    st, off, _ = oracle.scan_offsets(d, bits, meta, group)
    assert st == oracle.OK and payload.size == off[-1]
    for t in range(T):
        rec = payload[off[t]:off[t + 1]]
        b = int(bits[t])
        if b == 16:
            assert np.array_equal(rec.view("<u2"), x[t].view(np.uint16))
            continue
        G = d // group
        pairs = _pairs_bytes(d, meta, group)
        assert np.all(rec[meta * G:pairs] == 0)
        codes = []
        for g in range(G):
            s, z, q = oracle.quantize_span(x[t, group * g:group * (g + 1)], b, compact=(meta == 4))
            if meta == 8:
                assert rec[8 * g:8 * g + 8].view("<f4").tolist() == [float(s), float(z)]
            else:
                assert rec[4 * g:4 * g + 4].view("<f2").tolist() == [float(s), float(z)]
            codes.append(q)
        allq = np.concatenate(codes)
        bitstring = np.unpackbits(allq[:, None], axis=1, bitorder="little")[:, :b].reshape(-1)
        assert np.array_equal(rec[pairs:], np.packbits(bitstring, bitorder="little"))
    back = oracle.decode_stream(payload, bits, d, meta, group)
    assert np.array_equal(back[3].view(np.uint16), x[3].view(np.uint16))


@pytest.mark.parametrize("group,meta,d", [(64, 8, 128), (128, 4, 128), (128, 8, 256), (64, 4, 256)])
def test_whole_card_round_trip_and_header(group, meta, d):
    L, H, T = 2, 2, 70
    rng = np.random.default_rng(group + meta + d)
    Ks = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16) for _ in range(L)]
    Vs = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16) for _ in range(L)]
    bits = wl.iid_bits(T, (0.3, 0.3, 0.3, 0.1), 5)
    lay = oracle.make_layout(L, H, d, T, meta_bytes=meta, group_size=group)
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    hd = oracle.parse_header(card)
    assert hd["group_size"] == group and hd["meta_bytes_per_group"] == meta
    per_stream = sum(oracle.record_bytes(d, int(b), meta, group) for b in bits)
    assert hd["stream_bytes"] == per_stream and card.size == hd["payload_off"] + 2 * L * H * per_stream
    for s, arr in ((0, Ks[0][0]), (H, Vs[0][0]), (2 * H + 1, Ks[1][1])):
        a = hd["payload_off"] + s * per_stream
        assert np.array_equal(card[a:a + per_stream], oracle.encode_stream(arr, bits, meta, group))
    Ko, Vo = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, lay, Ko, Vo) == oracle.OK
    want = oracle.decode_stream(oracle.encode_stream(Vs[1][0], bits, meta, group), bits, d, meta, group)
    assert np.array_equal(Vo[1][0].view(np.uint16), want.view(np.uint16))
    # a card is read back with the group size it was made with
    other = oracle.make_layout(L, H, d, T, meta_bytes=meta, group_size=32 if group != 32 else 64)
    if not (meta == 4 and d % 128):
        assert oracle.card_inject(card, other, Ko, Vo) == oracle.BAD_CARD


def test_attention_over_a_wide_group_card_is_library_attention_on_its_injected_cache():
    L, H, d, T, nq = 1, 2, 128, 90, 4
    rng = np.random.default_rng(3)
    Ks = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16)]
    Vs = [rng.standard_normal((H, T, d), dtype=np.float32).astype(np.float16)]
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 4)
    lay = oracle.make_layout(L, H, d, T, group_size=64)
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    Kr, Vr = [np.zeros_like(Ks[0])], [np.zeros_like(Vs[0])]
    assert oracle.card_inject(card, lay, Kr, Vr) == oracle.OK
    q = wl.random_fp16((L, nq, d), 5)
    st, o = oracle.card_attend(card, lay, q, injected=True)
    assert st == oracle.OK
    for j in range(nq):
        k, v = Kr[0][j // 2].astype(np.float64), Vr[0][j // 2].astype(np.float64)
        s = k @ q[0, j].astype(np.float64) / np.sqrt(d)
        p = np.exp(s - s.max())
        np.testing.assert_allclose(o[0, j], (p / p.sum()) @ v, rtol=1e-12, atol=1e-14)
    st, o2 = oracle.card_attend(card, lay, q)
    assert st == oracle.OK and 0 < np.abs(o2 - o).max() < 2.0 ** -9 * np.abs(Vr[0].astype(np.float64)).max()
