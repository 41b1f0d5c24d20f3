"""Pins for the oracle's compact-metadata card variant (FP16 scale rounded up + FP16 zero, 4 bytes
per group).  The paper's "about 0.5 bytes per element at 4 bits" (Section 3.1) is only approached
as the per-group metadata shrinks; the variant's arithmetic is a reading, so it is pinned here by
hand-worked groups, a brute-force search over every FP16 value, exact rational recomputation, the
error bound the rounding direction guarantees, and special cases that reduce to the fp32-metadata
format.  None of the checks below calls the CUDA library.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from golden_io import read_fixture


def _h_bits(h) -> int:
    return int(np.float16(h).view(np.uint16))


def _groups(seed, n, spread=1.0, outlier=False):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, 32), dtype=np.float32) * np.float32(spread)
    if outlier:
        x[:, 5] *= 10
    return x.astype(np.float16)


_POS_HALVES = np.arange(0, 0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)  # ascending


def _half_up_brute(f: float) -> int:
    """Bit pattern of the smallest non-negative FP16 value >= f, by search over all of them."""
    return int(np.searchsorted(_POS_HALVES, np.float64(f), side="left"))


# ----------------------------------------------------------------------------- sizes

def test_compact_record_bytes_closed_form_fixture():
    fx = read_fixture("card_sizes.txt")
    for d, b, n in fx["crec"]:
        assert oracle.record_bytes(int(d), int(b), 4) == int(n)
    for b in (0, 1, 3, 5, 12, 17, 255):
        assert oracle.record_bytes(128, b, 4) == -1
    for meta in (0, 2, 6, 16):
        assert oracle.record_bytes(128, 4, meta) == -1


def test_effective_bits_per_element():
    """4 bytes per 32 elements add exactly one bit per element: 3 / 5 / 9 bits at 2 / 4 / 8."""
    for d in (128, 256):
        for b in (2, 4, 8):
            assert Fraction(8 * oracle.record_bytes(d, b, 4), d) == b + 1
            assert Fraction(8 * oracle.record_bytes(d, b, 8), d) == b + 2
        assert oracle.record_bytes(d, 16, 4) == oracle.record_bytes(d, 16, 8) == 2 * d


def test_compact_card_size_closed_form_fixture():
    fx = read_fixture("card_sizes.txt")
    for L, H, d, T, c16, c8, c4, c2, payload in fx["cpayload"]:
        L, H, d, T = int(L), int(H), int(d), int(T)
        bits = np.concatenate([np.full(int(c16), 16), np.full(int(c8), 8), np.full(int(c4), 4),
                               np.full(int(c2), 2)]).astype(np.uint8)
        np.random.default_rng(0).shuffle(bits)
        st, total = oracle.card_size(oracle.make_layout(L, H, d, T, meta_bytes=4), bits)
        assert st == oracle.OK
        a = lambda x: (x + 255) // 256 * 256
        assert total == 256 + a(T) + a(4 * (T + 1)) + int(payload)


def test_compact_needs_head_dim_multiple_of_128():
    """Records must stay multiples of 16 bytes: d = 64 would give 24-byte 2-bit records."""
    for d in (64, 192):
        st, _ = oracle.card_size(oracle.make_layout(1, 1, d, 8, meta_bytes=4), None)
        assert st == oracle.UNSUPPORTED_SHAPE
    for d in (128, 256):
        st, _ = oracle.card_size(oracle.make_layout(1, 1, d, 8, meta_bytes=4), None)
        assert st == oracle.OK
        for b in (2, 4, 8, 16):
            assert oracle.record_bytes(d, b, 4) % 16 == 0
    st, _ = oracle.card_size(oracle.make_layout(1, 1, 128, 8, meta_bytes=2), None)
    assert st == oracle.INVALID_ARG


def test_compact_offsets_equal_library_cumsum():
    rng = np.random.default_rng(3)
    bits = rng.choice(np.array([2, 4, 8, 16], np.uint8), size=1000)
    st, off, sb = oracle.scan_offsets(128, bits, 4)
    assert st == oracle.OK and sb == int(bits.astype(np.int64).sum())
    rec = {2: 48, 4: 80, 8: 144, 16: 256}
    assert off.tolist() == np.concatenate([[0], np.cumsum([rec[int(b)] for b in bits])]).tolist()


# ----------------------------------------------------------------------------- rounding up to FP16

def test_round_up_to_half_against_search_over_all_halves():
    rng = np.random.default_rng(11)
    vals = np.concatenate([
        rng.random(4000, dtype=np.float32) * np.float32(4.0),
        np.exp(rng.uniform(np.log(1e-9), np.log(43000.0), 4000)).astype(np.float32),
        _POS_HALVES[::37].astype(np.float32),                       # exact FP16 values stay put
        np.nextafter(_POS_HALVES[1::41].astype(np.float32), np.float32(0)),   # just below one
        np.nextafter(_POS_HALVES[:-1:43].astype(np.float32), np.float32(1e9)),  # just above one
        np.array([0.0, 2.0 ** -25, 2.0 ** -24, 2.0 ** -24 / 255, 43669.332, 65504.0], np.float32)])
    for f in vals:
        assert oracle.float_to_half_up(float(f)) == _half_up_brute(float(f)), float(f)


# ----------------------------------------------------------------------------- worked examples

@pytest.mark.parametrize("name", ["compact_example_d_2bit.txt", "compact_example_e_4bit.txt"])
def test_compact_worked_examples(name):
    fx = read_fixture(name)
    b = int(fx["bits"][0][0])
    x = np.array([float(v) for v in fx["x"][0]], dtype=np.float16)
    assert np.array_equal(x.astype(np.float64), [float(v) for v in fx["x"][0]])
    scale, zero, q = oracle.quantize_group_compact(x, b)
    assert _h_bits(scale) == int(fx["scale_bits"][0][0], 16)
    assert _h_bits(zero) == int(fx["zero_bits"][0][0], 16)
    assert q.tolist() == [int(v) for v in fx["codes"][0]]
    assert oracle.pack_codes(q, b).tolist() == [int(v, 16) for v in fx["packed_hex"][0]]
    deq = oracle.dequantize_group(q, np.float32(scale), np.float32(zero))
    assert deq.astype(np.float64).tolist() == [float(v) for v in fx["dequant"][0]]
    # through the record path: G = 4 groups -> 4 {scale, zero} FP16 pairs (16 bytes), then codes
    row = np.tile(x, 4)[None, :]
    rec = oracle.encode_stream(row, np.array([b], np.uint8), 4)
    assert rec.size == oracle.record_bytes(128, b, 4)
    assert rec[:16].view("<u2").tolist() == [int(fx["scale_bits"][0][0], 16),
                                             int(fx["zero_bits"][0][0], 16)] * 4
    assert rec[16:].tolist() == [int(v, 16) for v in fx["packed_hex"][0]] * 4
    back = oracle.decode_stream(rec, np.array([b], np.uint8), 128, 4)
    assert back.astype(np.float64)[0].tolist() == [float(v) for v in fx["dequant"][0]] * 4


def test_example_d_differs_from_fp32_metadata_exactly_where_worked():
    """With fp32 metadata 0.5 sits on the tie 1.5 and goes to code 2; with the rounded-up FP16
    scale it is below the tie and goes to 1.  Codes follow the stored scale."""
    fx = read_fixture("compact_example_d_2bit.txt")
    x = np.array([float(v) for v in fx["x"][0]], dtype=np.float16)
    _, _, q8 = oracle.quantize_group(x, 2)
    _, _, q4 = oracle.quantize_group_compact(x, 2)
    differ = np.nonzero(q8 != q4)[0]
    assert differ.tolist() == [2, 10, 18, 26] and set(x[differ].tolist()) == {0.5}
    assert q8[2] == 2 and q4[2] == 1


# ----------------------------------------------------------------------------- properties

def _rn32(fr: Fraction) -> Fraction:
    """Correctly rounded (nearest-even) binary32 value of a rational, in rational arithmetic."""
    if fr == 0:
        return Fraction(0)
    s = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    e = max(e, -126)
    ulp = Fraction(2) ** (e - 23)
    n = a / ulp
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return s * fl * ulp


@pytest.mark.parametrize("b", [2, 4, 8])
def test_compact_step_by_step_in_rationals(b):
    """Every step rounded once, in exact rational arithmetic, with the round-up done by search
    over all FP16 values: reproduces scale, zero, codes and reconstruction bit for bit."""
    qmax = (1 << b) - 1
    for x in np.concatenate([_groups(41, 25), _groups(42, 15, 40.0), _groups(43, 10, 1e-3),
                             _groups(44, 10, outlier=True)]):
        scale, zero, q = oracle.quantize_group_compact(x, b)
        fx = [Fraction(float(v)) for v in x]
        mn, mx = min(fx), max(fx)
        assert Fraction(float(zero)) == mn
        rng_ = _rn32(mx - mn)
        s32 = _rn32(rng_ / qmax)
        s16 = Fraction(float(_POS_HALVES[_half_up_brute(float(s32))]))
        assert Fraction(float(scale)) == s16
        inv = _rn32(1 / s16)
        deq = oracle.dequantize_group(q, np.float32(scale), np.float32(zero))
        for i in range(32):
            u = _rn32(_rn32(fx[i] - mn) * inv)
            fl = u.numerator // u.denominator
            rem = u - fl
            code = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2) else 0)
            assert int(q[i]) == min(code, qmax)
            r = _rn32(_rn32(int(q[i]) * s16) + mn)
            assert float(deq[i]) == float(np.float32(float(r)).astype(np.float16))


@pytest.mark.parametrize("b", [2, 4, 8])
def test_compact_scale_bounds_and_error(b):
    """The stored scale is at least range/(2^b-1) (up to the fp32 rounding of that quotient) and
    less than one FP16 step above it; min -> code 0 and reconstructs exactly; max -> the top code
    or, when the round-up leaves it under the last tie, the one below; codes are monotone;
    |x - x^| <= scale/2 plus rounding slack."""
    qmax = (1 << b) - 1
    for x in np.concatenate([_groups(51, 300), _groups(52, 300, 30.0), _groups(53, 200, 1e-2),
                             _groups(54, 200, outlier=True)]):
        scale, zero, q = oracle.quantize_group_compact(x, b)
        xf = x.astype(np.float64)
        rng_ = xf.max() - xf.min()
        s = float(scale)
        assert s >= rng_ / qmax * (1 - 2.0 ** -23)
        assert s <= rng_ / qmax * (1 + 2.0 ** -23) + float(np.spacing(np.float16(s)))
        assert float(zero) == xf.min()
        assert q[np.argmin(xf)] == 0 and q.max() <= qmax
        assert q[np.argmax(xf)] >= qmax - 1
        order = np.argsort(xf, kind="stable")
        assert np.all(np.diff(q[order].astype(np.int32)) >= 0)
        deq = oracle.dequantize_group(q, np.float32(scale), np.float32(zero)).astype(np.float64)
        assert deq[np.argmin(xf)] == xf.min()
        ulp16 = np.abs(np.spacing(deq.astype(np.float16))).astype(np.float64)
        big = max(abs(xf.min()), abs(xf.max()))
        slack = 0.5 * ulp16 + 4 * float(np.spacing(np.float32(big))) + qmax * s * 2.0 ** -22
        assert np.all(np.abs(xf - deq) <= s / 2 + slack)


def test_compact_equals_fp32_format_when_the_scale_is_an_fp16_value():
    """Ranges of qmax * 2^k make range/qmax a power of two: the round-up is the identity and
    1/scale is exact, so codes and reconstructions equal the fp32-metadata format's."""
    rng = np.random.default_rng(61)
    for b in (2, 4, 8):
        qmax = (1 << b) - 1
        for k in (-6, -3, 0, 2):
            step = 2.0 ** k
            base = float(rng.integers(-20, 20)) * step
            codes = rng.integers(0, qmax + 1, 32)
            codes[0], codes[1] = 0, qmax
            x = (base + codes * step).astype(np.float16)
            assert np.array_equal(x.astype(np.float64), base + codes * step)
            s8, z8, q8 = oracle.quantize_group(x, b)
            s4, z4, q4 = oracle.quantize_group_compact(x, b)
            assert float(s4) == float(s8) == step and float(z4) == float(z8) == base
            assert q4.tolist() == q8.tolist() == codes.tolist()


def test_compact_constant_group_and_signed_zero():
    for v in (0.0, -0.0, 1.25, -3.5, 65504.0, 6e-8):
        x = np.full(32, v, dtype=np.float16)
        for b in (2, 4, 8):
            scale, zero, q = oracle.quantize_group_compact(x, b)
            assert _h_bits(scale) == 0 and not q.any()
            deq = oracle.dequantize_group(q, np.float32(scale), np.float32(zero))
            assert np.array_equal(deq.astype(np.float32), x.astype(np.float32))
    x = np.zeros(32, dtype=np.float16)
    x[::2] = -0.0
    x[3] = 2.0
    for b in (2, 4, 8):
        scale, zero, q = oracle.quantize_group_compact(x, b)
        assert _h_bits(zero) == 0
        assert q[3] >= (1 << b) - 2 and q.sum() == q[3]


def test_compact_extreme_magnitudes():
    """Largest range: scale = 131008/3 rounded up stays finite; smallest: one FP16 subnormal step
    at 8 bits gives scale = 2^-24 (the smallest FP16 value), codes 0 and 1."""
    x = np.zeros(32, dtype=np.float16)
    x[0], x[1] = -65504.0, 65504.0
    scale, zero, q = oracle.quantize_group_compact(x, 2)
    assert np.isfinite(np.float32(scale)) and float(scale) >= 131008.0 / 3
    assert _h_bits(scale) == _half_up_brute(float(np.float32(131008.0) / np.float32(3.0)))
    assert q[0] == 0 and q[1] == 3 and float(zero) == -65504.0
    y = np.zeros(32, dtype=np.float16)
    y[7] = np.float16(2.0 ** -24)
    scale, zero, q = oracle.quantize_group_compact(y, 8)
    assert _h_bits(scale) == 1 and _h_bits(zero) == 0
    assert q[7] == 1 and q.sum() == 1
    deq = oracle.dequantize_group(q, np.float32(scale), np.float32(zero))
    assert np.array_equal(deq, y)


# ----------------------------------------------------------------------------- whole cards

def _cache(L, H, T, d, seed):
    rng = np.random.default_rng(seed)
    Ks = [(rng.standard_normal((H, T, d), dtype=np.float32) * 2).astype(np.float16) for _ in range(L)]
    Vs = [(rng.standard_normal((H, T, d), dtype=np.float32) * 2).astype(np.float16) for _ in range(L)]
    return Ks, Vs


def test_compact_card_header_streams_and_round_trip():
    L, H, T, d = 2, 2, 37, 128
    Ks, Vs = _cache(L, H, T, d, 71)
    bits = np.random.default_rng(72).choice(np.array([2, 4, 8, 16], np.uint8), size=T)
    lay = oracle.make_layout(L, H, d, T, meta_bytes=4)
    st, card = oracle.card_create(lay, Ks, Vs, bits, model_id=5, sender_id=6)
    assert st == oracle.OK
    hdr = oracle.parse_header(card)
    assert hdr["meta_bytes_per_group"] == 4 and hdr["status"] == 0
    _, off, _ = oracle.scan_offsets(d, bits, 4)
    assert hdr["stream_bytes"] == int(off[-1])
    assert hdr["total_bytes"] == card.size == hdr["payload_off"] + 2 * L * H * int(off[-1])
    # every stream is the stream encoder's output, in (layer, K|V, head) order
    for l in range(L):
        for kv, src in enumerate((Ks, Vs)):
            for h in range(H):
                s = (l * 2 + kv) * H + h
                a = hdr["payload_off"] + s * int(off[-1])
                assert np.array_equal(card[a:a + int(off[-1])], oracle.encode_stream(src[l][h], bits, 4))
    Ko = [np.zeros((H, T, d), np.float16) for _ in range(L)]
    Vo = [np.zeros((H, T, d), np.float16) for _ in range(L)]
    assert oracle.card_inject(card, lay, Ko, Vo) == oracle.OK
    fp = bits == 16
    for l in range(L):
        assert np.array_equal(Ko[l][:, fp].view(np.uint16), Ks[l][:, fp].view(np.uint16))
        for h in range(H):
            assert np.array_equal(Vo[l][h], oracle.decode_stream(
                oracle.encode_stream(Vs[l][h], bits, 4), bits, d, 4))
    # a receiver that expects the other metadata format refuses the card
    lay8 = oracle.make_layout(L, H, d, T)
    assert oracle.card_inject(card, lay8, Ko, Vo) == oracle.BAD_CARD
    st8, card8 = oracle.card_create(lay8, Ks, Vs, bits)
    assert st8 == oracle.OK and oracle.card_inject(card8, lay, Ko, Vo) == oracle.BAD_CARD


def test_all_fp16_compact_card_equals_fp32_format_card_but_for_the_header_field():
    L, H, T, d = 1, 2, 19, 128
    Ks, Vs = _cache(L, H, T, d, 73)
    bits = np.full(T, 16, np.uint8)
    st4, c4 = oracle.card_create(oracle.make_layout(L, H, d, T, meta_bytes=4), Ks, Vs, bits)
    st8, c8 = oracle.card_create(oracle.make_layout(L, H, d, T), Ks, Vs, bits)
    assert st4 == st8 == oracle.OK and c4.size == c8.size
    diff = np.nonzero(c4 != c8)[0]
    assert diff.tolist() == [36] and c4[36] == 4 and c8[36] == 8


def test_attention_from_a_compact_card_matches_numpy_on_decoded_records():
    """Tiny case by brute force: rebuild K~, V~ in float64 from the record bytes with numpy
    (FP16 pair widened, code * scale + zero, no FP16 rounding) and apply the softmax definition."""
    L, H, T, d, nq = 1, 2, 9, 128, 4
    Ks, Vs = _cache(L, H, T, d, 75)
    bits = np.array([2, 4, 8, 16, 4, 2, 8, 4, 16], np.uint8)
    lay = oracle.make_layout(L, H, d, T, meta_bytes=4)
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    q = (np.random.default_rng(76).standard_normal((L, nq, d)) * 0.5).astype(np.float16)
    st, out = oracle.card_attend(card, lay, q)
    assert st == oracle.OK
    hdr = oracle.parse_header(card)
    _, off, _ = oracle.scan_offsets(d, bits, 4)

    def rebuild(stream):
        rows = np.zeros((T, d))
        for t in range(T):
            rec = stream[off[t]:off[t + 1]]
            b = int(bits[t])
            if b == 16:
                rows[t] = rec.view("<f2").astype(np.float64)
                continue
            meta = rec[:16].view("<f2").astype(np.float64)
            bitstr = np.unpackbits(rec[16:], bitorder="little").reshape(d, b)
            codes = (bitstr * (1 << np.arange(b))).sum(axis=1).astype(np.float64)
            rows[t] = codes * np.repeat(meta[0::2], 32) + np.repeat(meta[1::2], 32)
        return rows

    for h in range(H):
        base = hdr["payload_off"]
        kx = rebuild(card[base + (0 * H + h) * int(off[-1]):][:int(off[-1])])
        vx = rebuild(card[base + (1 * H + h) * int(off[-1]):][:int(off[-1])])
        for jj in range(nq // H):
            j = h * (nq // H) + jj
            s = kx @ q[0, j].astype(np.float64) / np.sqrt(d)
            p = np.exp(s - s.max())
            p /= p.sum()
            assert np.allclose(out[0, j], p @ vx, rtol=1e-12, atol=1e-12)
