"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without the GPU.

Each test states what independent fact it pins.  None of them re-types the oracle's
arithmetic: they use closed forms, hand-worked fixtures, invariants, exact rational
arithmetic, numpy library routines for the special cases that reduce to one, and brute force.
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from golden_io import read_fixture
from rank_rule import by_library_sort
from paper_2605_03884_b200 import workloads as wl


def _f32_bits(x) -> int:
    return int(np.float32(x).view(np.uint32))


def _groups(seed, n, spread=1.0, outlier=False):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, 32), dtype=np.float32) * np.float32(spread)
    if outlier:
        x[:, 5] *= 10
    return x.astype(np.float16)


# ----------------------------------------------------------------------------- FP16 conversion

def test_half_to_float_all_patterns_match_numpy():
    """Every FP16 bit pattern converts to the value numpy's float16 gives (library routine)."""
    pats = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = pats.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(p)) for p in pats], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_float_to_half_matches_numpy_rne():
    """Round-to-nearest-even to FP16, including ties, subnormals and overflow (numpy routine)."""
    rng = np.random.default_rng(7)
    vals = [0.0, -0.0, 1.0, 65504.0, 65519.99, 65520.0, 70000.0, -65520.0, 2.0 ** -14, 2.0 ** -24,
            2.0 ** -25, 2.0 ** -25 * 1.0000001, 3 * 2.0 ** -25, 2.0 ** -14 - 2.0 ** -25,
            1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2047.5, 2048.5, 1e-10, float("inf")]
    vals += list(rng.standard_normal(20000) * 3)
    vals += list(rng.standard_normal(5000) * 1e-5)
    vals += list(rng.standard_normal(5000) * 3e4)
    # exact ties between neighbouring FP16 values
    h = rng.integers(0, 0x7bff, 5000).astype(np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    vals += list((lo + hi) / 2)
    a = np.array(vals, dtype=np.float32)
    with np.errstate(over="ignore"):
        want = a.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(float(v)) for v in a], dtype=np.uint16)
    assert np.array_equal(got, want)


# ----------------------------------------------------------------------------- sizes, offsets

def test_record_bytes_closed_form_fixture():
    fx = read_fixture("card_sizes.txt")
    for d, b, n in fx["rec"]:
        assert oracle.record_bytes(int(d), int(b)) == int(n)
    for b in (0, 1, 3, 5, 6, 7, 12, 15, 17, 32, 255):
        assert oracle.record_bytes(128, b) == -1


def test_code_bytes_follow_bytes_per_element_law():
    """Section 3.1: FP16 is 2 B/element, 4-bit is 0.5 B/element (4x) once metadata is set aside."""
    for d in (64, 128, 256):
        meta = 8 * (d // 32)
        assert oracle.record_bytes(d, 16) == 2 * d
        assert oracle.record_bytes(d, 4) - meta == d // 2
        assert (2 * d) / (oracle.record_bytes(d, 4) - meta) == 4.0
        assert oracle.record_bytes(d, 2) - meta == d // 4
        assert oracle.record_bytes(d, 8) - meta == d


def test_card_size_closed_form_fixture():
    fx = read_fixture("card_sizes.txt")
    for L, H, d, T, c16, c8, c4, c2, payload in fx["payload"]:
        L, H, d, T = int(L), int(H), int(d), int(T)
        bits = np.concatenate([np.full(int(c16), 16), np.full(int(c8), 8), np.full(int(c4), 4),
                               np.full(int(c2), 2)]).astype(np.uint8)
        np.random.default_rng(0).shuffle(bits)
        assert bits.size == T
        st, total = oracle.card_size(oracle.make_layout(L, H, d, T), bits)
        assert st == oracle.OK
        a = lambda x: (x + 255) // 256 * 256
        assert total == 256 + a(T) + a(4 * (T + 1)) + int(payload)


def test_quantile_bits_counts_match_fixture():
    """The 8K adaptive recipe gives the 410 / 1228 / 3277 / 3277 split the size fixture assumes."""
    bits = wl.bits_for(wl.WORKLOADS[4], rank_rule=by_library_sort)
    assert [int((bits == b).sum()) for b in (16, 8, 4, 2)] == [410, 1228, 3277, 3277]


def test_card_size_worst_case_and_errors():
    lay = oracle.make_layout(2, 2, 64, 10)
    st, worst = oracle.card_size(lay, None)
    st2, allfp = oracle.card_size(lay, np.full(10, 16, np.uint8))
    assert st == st2 == oracle.OK and worst == allfp
    assert oracle.card_size(lay, np.array([4] * 9 + [3], np.uint8))[0] == oracle.BAD_BITS
    assert oracle.card_size(oracle.make_layout(1, 1, 32, 4), None)[0] == oracle.UNSUPPORTED_SHAPE
    assert oracle.card_size(oracle.make_layout(1, 1, 96, 4), None)[0] == oracle.UNSUPPORTED_SHAPE
    bad = oracle.make_layout(1, 1, 64, 4)
    bad.group_size = 48
    assert oracle.card_size(bad, None)[0] == oracle.UNSUPPORTED_SHAPE


@pytest.mark.parametrize("d", [64, 128])
def test_uniform_offsets_are_multiples_of_record(d):
    for b in (2, 4, 8, 16):
        st, off, sb = oracle.scan_offsets(d, np.full(777, b, np.uint8))
        assert st == oracle.OK and sb == 777 * b
        assert np.array_equal(off, np.arange(778, dtype=np.uint64) * oracle.record_bytes(d, b))


def test_offsets_equal_library_cumsum():
    """Exclusive prefix sum == numpy.cumsum over a lookup of record sizes."""
    rng = np.random.default_rng(3)
    for d in (64, 128, 256):
        bits = wl.BIT_CHOICES[rng.integers(0, 4, 5000)]
        lut = np.zeros(17, dtype=np.int64)
        for b in (2, 4, 8, 16):
            lut[b] = oracle.record_bytes(d, b)
        want = np.concatenate([[0], np.cumsum(lut[bits])])
        st, off, sb = oracle.scan_offsets(d, bits)
        assert st == oracle.OK
        assert np.array_equal(off.astype(np.int64), want)
        assert sb == int(bits.astype(np.int64).sum())
        assert np.all(off % 16 == 0)          # every record starts on a 16-byte boundary


def test_scan_rejects_bad_bits():
    for bad in (0, 1, 3, 5, 6, 7, 9, 15, 17, 32, 255):
        bits = np.full(50, 4, np.uint8)
        bits[17] = bad
        assert oracle.scan_offsets(128, bits)[0] == oracle.BAD_BITS


# ----------------------------------------------------------------------------- worked examples

@pytest.mark.parametrize("name", ["worked_example_a_4bit.txt", "worked_example_b_2bit.txt",
                                  "worked_example_c_8bit.txt"])
def test_worked_examples(name):
    """Hand-worked groups with exact ties: pins rounding mode, scale/zero, packing order, dequant."""
    fx = read_fixture(name)
    b = int(fx["bits"][0][0])
    x = np.array([float(v) for v in fx["x"][0]], dtype=np.float16)
    assert np.array_equal(x.astype(np.float64), [float(v) for v in fx["x"][0]])  # exactly FP16
    scale, zero, q = oracle.quantize_group(x, b)
    assert _f32_bits(scale) == int(fx["scale_bits"][0][0], 16)
    assert _f32_bits(zero) == int(fx["zero_bits"][0][0], 16)
    assert q.tolist() == [int(v) for v in fx["codes"][0]]
    packed = oracle.pack_codes(q, b)
    assert packed.tolist() == [int(v, 16) for v in fx["packed_hex"][0]]
    assert oracle.unpack_codes(packed, 32, b).tolist() == q.tolist()
    deq = oracle.dequantize_group(q, scale, zero)
    assert deq.astype(np.float64).tolist() == [float(v) for v in fx["dequant"][0]]
    # the same group through the whole record path: metadata first, then codes
    rec = oracle.encode_stream(np.tile(x, 2)[None, :], np.array([b], np.uint8))
    meta = rec[:16].view("<u4")
    assert meta.tolist() == [int(fx["scale_bits"][0][0], 16), int(fx["zero_bits"][0][0], 16)] * 2
    assert rec[16:].tolist() == [int(v, 16) for v in fx["packed_hex"][0]] * 2


def test_worked_example_with_an_inexact_scale():
    """A group whose range / qmax is not a binary32 value, at 4, 2 and 8 bits: the stored figures
    (worked in rationals, see the fixture's header) against the oracle, and against a fresh
    recomputation in exact rational arithmetic here, so that the fixture itself is checked."""
    fx = read_fixture("worked_example_f_inexact.txt")
    x = np.array([int(v) for v in fx["x_bits"][0]], dtype=np.uint16)
    xf = [_frac16(v) for v in x.view(np.float16)]
    mn, mx = min(xf), max(xf)
    assert mx - mn == Fraction(4097, 1024) and xf.index(mn) == 20 and xf.index(mx) == 7
    for (b, scale_hex, inv_hex), codes, packed in zip(fx["case"], fx["codes"], fx["packed_hex"]):
        b, qmax = int(b), (1 << int(b)) - 1
        want_codes = [int(v) for v in codes]
        sc, inv = _rn32((mx - mn) / qmax), _rn32(Fraction(qmax) / (mx - mn))
        assert _f32_bits(np.float32(float(sc))) == int(scale_hex, 16)
        assert _f32_bits(np.float32(float(inv))) == int(inv_hex, 16)
        for v, c in zip(xf, want_codes):
            u = _rn32(_rn32(v - mn) * inv)
            fl = u.numerator // u.denominator
            rem = u - fl
            assert c == min(fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2) else 0), qmax)
        bitstring = sum(c << (i * b) for i, c in enumerate(want_codes))
        assert list(bitstring.to_bytes(4 * b, "little")) == [int(v, 16) for v in packed]
        scale, zero, q = oracle.quantize_group(x, b)
        assert _f32_bits(scale) == int(scale_hex, 16) and _f32_bits(zero) == int(fx["zero_bits"][0][0], 16)
        assert q.tolist() == want_codes
        assert oracle.pack_codes(q, b).tolist() == [int(v, 16) for v in packed]
        deq = oracle.dequantize_group(q, scale, zero).astype(np.float64)
        assert np.abs(deq - np.array([float(v) for v in xf])).max() <= float(sc) / 2 + 2.0 ** -11 * 2.5


def test_pack_order_matches_little_endian_bitstream():
    """Packing == numpy's little-endian bit string of the codes (library routine)."""
    rng = np.random.default_rng(11)
    for b in (2, 4, 8):
        q = rng.integers(0, 1 << b, 128).astype(np.uint8)
        bitsarr = ((q[:, None] >> np.arange(b)) & 1).astype(np.uint8).reshape(-1)
        want = np.packbits(bitsarr, bitorder="little")
        assert np.array_equal(oracle.pack_codes(q, b), want)
        assert np.array_equal(oracle.unpack_codes(want, 128, b), q)


# ----------------------------------------------------------------------------- quantiser invariants

@pytest.mark.parametrize("b", [2, 4, 8])
def test_min_max_codes_monotone_and_min_exact(b):
    qmax = (1 << b) - 1
    for x in np.concatenate([_groups(1, 300), _groups(2, 300, 30.0), _groups(3, 200, 1e-3),
                             _groups(4, 200, outlier=True)]):
        scale, zero, q = oracle.quantize_group(x, b)
        xf = x.astype(np.float32)
        assert zero == xf.min()
        assert q[np.argmin(xf)] == 0 and q[np.argmax(xf)] == qmax
        assert q.max() <= qmax
        order = np.argsort(xf, kind="stable")
        assert np.all(np.diff(q[order].astype(np.int32)) >= 0)      # codes monotone in x
        deq = oracle.dequantize_group(q, scale, zero)
        assert deq[np.argmin(xf)] == x.min()                        # min reconstructs exactly


@pytest.mark.parametrize("b", [2, 4, 8])
def test_reconstruction_error_within_half_scale(b):
    """|x - x^| <= scale/2 in exact arithmetic; slack for the fp32 steps and the FP16 rounding."""
    for x in np.concatenate([_groups(5, 400), _groups(6, 300, 100.0), _groups(7, 300, 1e-2),
                             _groups(8, 300, outlier=True)]):
        scale, zero, q = oracle.quantize_group(x, b)
        deq = oracle.dequantize_group(q, scale, zero).astype(np.float64)
        xf = x.astype(np.float64)
        ulp16 = np.abs(np.spacing(deq.astype(np.float16))).astype(np.float64)
        big = max(abs(xf.min()), abs(xf.max()))
        slack = 0.5 * ulp16 + 4 * float(np.spacing(np.float32(big)))
        assert np.all(np.abs(xf - deq) <= float(scale) / 2 + slack)


def test_constant_group_and_signed_zero():
    for v in (0.0, -0.0, 1.25, -3.5, 65504.0, 6e-8):
        x = np.full(32, v, dtype=np.float16)
        for b in (2, 4, 8):
            scale, zero, q = oracle.quantize_group(x, b)
            assert _f32_bits(scale) == 0 and not q.any()
            deq = oracle.dequantize_group(q, scale, zero)
            assert np.array_equal(deq.astype(np.float32), x.astype(np.float32))
    # a zero minimum is stored as +0 even when the data holds -0
    x = np.zeros(32, dtype=np.float16)
    x[::2] = -0.0
    x[3] = 2.0
    for b in (2, 4, 8):
        scale, zero, q = oracle.quantize_group(x, b)
        assert _f32_bits(zero) == 0
        assert q[3] == (1 << b) - 1 and q.sum() == q[3]


def test_extreme_magnitudes():
    x = np.zeros(32, dtype=np.float16)
    x[0], x[1] = -65504.0, 65504.0
    x[2:] = np.linspace(-60000, 60000, 30).astype(np.float16)
    for b in (2, 4, 8):
        scale, zero, q = oracle.quantize_group(x, b)
        assert zero == -65504.0 and q[0] == 0 and q[1] == (1 << b) - 1
        deq = oracle.dequantize_group(q, scale, zero)
        assert np.all(np.isfinite(deq.astype(np.float32)))
    sub = (np.arange(32, dtype=np.uint16) * 3).view(np.float16)   # subnormals, range 93 * 2^-24
    for b in (2, 4, 8):
        scale, zero, q = oracle.quantize_group(sub, b)
        assert zero == 0 and q[0] == 0 and q[31] == (1 << b) - 1
        assert np.all(np.diff(q.astype(int)) >= 0)


# ----------------------------------------------------------------------------- exact arithmetic

def _frac16(h) -> Fraction:
    return Fraction(float(np.float16(h)))


def _ulp16(mag: Fraction) -> Fraction:
    """Spacing of FP16 values in the binade that holds `mag` (subnormal spacing below 2^-14)."""
    e = -14
    while Fraction(2) ** (e + 1) <= mag:
        e += 1
    return Fraction(2) ** (e - 10)


@pytest.mark.parametrize("b", [2, 4, 8])
def test_codes_against_exact_rational_quantiser(b):
    """Exact u* = (x-min)*(2^b-1)/(max-min) over the rationals: the code is round(u*) unless u*
    sits within the fp32 rounding error of a tie, and the reconstruction is within half an FP16
    ulp (plus fp32 slack) of min + q*(max-min)/(2^b-1)."""
    qmax = (1 << b) - 1
    eps = Fraction(qmax, 1 << 21)          # three fp32 roundings on a value <= qmax
    groups = np.concatenate([_groups(21, 60), _groups(22, 40, 50.0), _groups(23, 40, outlier=True)])
    for x in groups:
        scale, zero, q = oracle.quantize_group(x, b)
        fx = [_frac16(v) for v in x]
        mn, mx = min(fx), max(fx)
        assert Fraction(float(zero)) == mn
        rng_ = mx - mn
        assert abs(Fraction(float(scale)) - rng_ / qmax) <= rng_ / qmax / (1 << 23)
        deq = oracle.dequantize_group(q, scale, zero)
        for i in range(32):
            u = (fx[i] - mn) * qmax / rng_
            lo, hi = u - Fraction(1, 2), u + Fraction(1, 2)
            assert lo - eps <= int(q[i]) <= hi + eps
            if abs((u % 1) - Fraction(1, 2)) > eps:
                assert int(q[i]) == round(u)
            xr = mn + int(q[i]) * rng_ / qmax
            d16 = _ulp16(max(abs(xr), abs(Fraction(float(deq[i])))))
            assert abs(Fraction(float(deq[i])) - xr) <= d16 / 2 + abs(xr) / (1 << 21) + rng_ / (1 << 21)


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
def test_step_by_step_ieee_emulation_in_rationals(b):
    """Each step rounded once to binary32 in exact rational arithmetic reproduces scale, codes and
    reconstruction bit for bit: catches fused operations, double rounding or excess precision in
    the compiled oracle."""
    qmax = (1 << b) - 1
    for x in np.concatenate([_groups(31, 25), _groups(32, 15, 40.0), _groups(33, 10, 1e-3)]):
        scale, zero, q = oracle.quantize_group(x, b)
        deq = oracle.dequantize_group(q, scale, zero)
        fx = [_frac16(v) for v in x]
        mn, mx = min(fx), max(fx)
        rng_ = _rn32(mx - mn)
        sc, inv = _rn32(rng_ / qmax), _rn32(Fraction(qmax) / rng_)
        assert Fraction(float(scale)) == sc
        for i in range(32):
            u = _rn32(_rn32(fx[i] - mn) * inv)
            fl = u.numerator // u.denominator
            rem = u - fl
            code = fl + (1 if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2) else 0)
            assert int(q[i]) == min(code, qmax)
            r = _rn32(_rn32(int(q[i]) * sc) + mn)
            assert float(deq[i]) == float(np.float32(float(r)).astype(np.float16))


def test_eight_bit_matches_textbook_affine_uint8():
    """One group at 8 bits == round((x-min)/(max-min)*255) computed in float64 (numpy), except
    where the exact value lies within 1e-4 of a tie."""
    for x in np.concatenate([_groups(41, 500), _groups(42, 300, 20.0)]):
        _, _, q = oracle.quantize_group(x, 8)
        xf = x.astype(np.float64)
        u = (xf - xf.min()) / (xf.max() - xf.min()) * 255.0
        clear = np.abs(u - np.floor(u) - 0.5) > 1e-4
        assert np.array_equal(q[clear], np.round(u[clear]).astype(np.uint8))
        assert np.all(np.abs(q.astype(np.float64) - u) <= 0.5 + 1e-4)


def test_requantising_a_reconstruction_keeps_min_and_max():
    """Repeated handoff (Section 6.1): a reconstructed group re-quantised at the same width keeps
    its extremes, so a second hop at equal width adds nothing beyond rounding."""
    for b in (2, 4, 8):
        for x in _groups(50 + b, 200):
            s1, z1, q1 = oracle.quantize_group(x, b)
            d1 = oracle.dequantize_group(q1, s1, z1)
            s2, z2, q2 = oracle.quantize_group(d1, b)
            d2 = oracle.dequantize_group(q2, s2, z2)
            assert z2 == z1
            assert d2.min() == d1.min() and d2.max() == d1.max()
            assert q2[np.argmax(d1.astype(np.float32))] == (1 << b) - 1


# ----------------------------------------------------------------------------- whole cards

def _cache(L, H, T, d, seed, t_cap=None, token_stride=None):
    """Per-layer K, V arrays (possibly padded) + the layout describing them."""
    t_cap = T if t_cap is None else t_cap
    ts = d if token_stride is None else token_stride
    rng = np.random.default_rng(seed)
    Ks, Vs = [], []
    for _ in range(L):
        for dst in (Ks, Vs):
            buf = np.full((H, t_cap, ts), 777.0, dtype=np.float16)
            buf[:, :T, :d] = (rng.standard_normal((H, T, d), dtype=np.float32) * 2).astype(np.float16)
            dst.append(buf)
    lay = oracle.make_layout(L, H, d, T, head_stride=t_cap * ts, token_stride=ts)
    return Ks, Vs, lay


def test_all_fp16_card_is_a_memcpy_in_stream_order():
    """With every token FP16 the payload is the cache itself, stream (l, K|V, h) after stream:
    pins stream order, strides and the FP16 pass-through."""
    L, H, T, d = 3, 2, 37, 64
    Ks, Vs, lay = _cache(L, H, T, d, 60, t_cap=50, token_stride=72)
    # plant special bit patterns: NaN payloads, infinities, -0, subnormals
    Ks[1].view(np.uint16)[1, 5, :8] = [0x7e01, 0xfe55, 0x7c00, 0xfc00, 0x8000, 0x0001, 0x83ff, 0x7dff]
    st, card = oracle.card_create(lay, Ks, Vs, np.full(T, 16, np.uint8))
    assert st == oracle.OK
    hd = oracle.parse_header(card)
    want = np.concatenate([a[h, :T, :d].reshape(-1).view(np.uint8)
                           for l in range(L) for a in (Ks[l], Vs[l]) for h in range(H)])
    assert hd["total_bytes"] == card.size == hd["payload_off"] + want.size
    assert np.array_equal(card[hd["payload_off"]:], want)
    # and back: inject reproduces every bit pattern
    Ko, Vo, dl = _cache(L, H, T, d, 61)
    assert oracle.card_inject(card, dl, Ko, Vo) == oracle.OK
    for l in range(L):
        assert np.array_equal(Ko[l].view(np.uint16), Ks[l][:, :T, :d].view(np.uint16))
        assert np.array_equal(Vo[l].view(np.uint16), Vs[l][:, :T, :d].view(np.uint16))


def test_fp16_tokens_round_trip_exactly_in_mixed_card():
    L, H, T, d = 2, 2, 96, 128
    Ks, Vs, lay = _cache(L, H, T, d, 62)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), 5)
    assert (bits == 16).sum() > 5
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    Ko, Vo, dl = _cache(L, H, T, d, 63)
    assert oracle.card_inject(card, dl, Ko, Vo) == oracle.OK
    m = bits == 16
    for l in range(L):
        assert np.array_equal(Ko[l][:, m].view(np.uint16), Ks[l][:, m].view(np.uint16))
        assert np.array_equal(Vo[l][:, m].view(np.uint16), Vs[l][:, m].view(np.uint16))
        assert not np.array_equal(Ko[l][:, ~m], Ks[l][:, ~m])


def test_header_fields_and_sections():
    L, H, T, d = 2, 3, 100, 64
    Ks, Vs, lay = _cache(L, H, T, d, 64)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 6)
    st, card = oracle.card_create(lay, Ks, Vs, bits, model_id=0x1122334455667788,
                                  sender_id=42, position_offset=-7)
    assert st == oracle.OK
    hd = oracle.parse_header(card)
    a = lambda x: (x + 255) // 256 * 256
    assert hd["magic"] == int.from_bytes(b"QKVS", "little") and hd["version"] == 1
    assert hd["status"] == 0 and hd["bits_mode"] == 0
    assert (hd["n_layers"], hd["n_kv_heads"], hd["head_dim"], hd["n_tokens"]) == (L, H, d, T)
    assert hd["group_size"] == 32 and hd["meta_bytes_per_group"] == 8
    assert hd["model_id"] == 0x1122334455667788 and hd["sender_id"] == 42
    assert hd["position_offset"] == -7
    assert hd["sum_bits"] == int(bits.astype(np.int64).sum())
    assert np.float32(hd["avg_code_bits"]) == np.float32(np.float32(hd["sum_bits"]) / np.float32(T))
    assert hd["bits_off"] == 256 and hd["offs_off"] == 256 + a(T)
    assert hd["payload_off"] == hd["offs_off"] + a(4 * (T + 1)) and hd["sbase_off"] == 0
    _, off, _ = oracle.scan_offsets(d, bits)
    assert hd["stream_bytes"] == int(off[-1])
    assert hd["total_bytes"] == card.size == oracle.card_size(lay, bits)[1]
    assert np.array_equal(card[256:256 + T], bits)
    assert np.array_equal(card[hd["offs_off"]:hd["offs_off"] + 4 * (T + 1)].view("<u4"), off)
    assert not card[120 + 8:256].any() and not card[256 + T:hd["offs_off"]].any()
    # each stream's slice is that stream encoded on its own
    for l in range(L):
        for kv, arr in enumerate((Ks[l], Vs[l])):
            for h in range(H):
                s = (l * 2 + kv) * H + h
                base = hd["payload_off"] + s * hd["stream_bytes"]
                assert np.array_equal(card[base:base + hd["stream_bytes"]],
                                      oracle.encode_stream(arr[h], bits))


def test_create_range_equals_slices_of_whole_card():
    L, H, T, d = 2, 2, 40, 64
    Ks, Vs, lay = _cache(L, H, T, d, 65)
    bits = wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 8)
    _, whole = oracle.card_create(lay, Ks, Vs, bits)
    _, part = oracle.card_create(lay, Ks, Vs, bits, streams=(3, 6))
    hd = oracle.parse_header(whole)
    sb, po = hd["stream_bytes"], hd["payload_off"]
    assert np.array_equal(part[:po], whole[:po])
    assert np.array_equal(part[po + 3 * sb:po + 6 * sb], whole[po + 3 * sb:po + 6 * sb])
    assert not part[po:po + 3 * sb].any() and not part[po + 6 * sb:].any()


def test_inject_with_offset_and_padded_destination():
    L, H, T, d = 2, 2, 33, 64
    Ks, Vs, lay = _cache(L, H, T, d, 66)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 9)
    _, card = oracle.card_create(lay, Ks, Vs, bits)
    Ko, Vo, dl = _cache(L, H, T, d, 67, t_cap=64, token_stride=80)
    before = [a.copy() for a in Ko]
    assert oracle.card_inject(card, dl, Ko, Vo, dst_token_offset=20) == oracle.OK
    for l in range(L):
        for h in range(H):
            want = oracle.decode_stream(oracle.encode_stream(Ks[l][h], bits), bits, d)
            assert np.array_equal(Ko[l][h, 20:20 + T, :d].view(np.uint16), want.view(np.uint16))
        untouched = np.ones_like(Ko[l], dtype=bool)
        untouched[:, 20:20 + T, :d] = False
        assert np.array_equal(Ko[l][untouched].view(np.uint16), before[l][untouched].view(np.uint16))
    assert oracle.card_inject(card, dl, Ko, Vo, dst_token_offset=32) == oracle.INVALID_ARG
    assert oracle.card_inject(card, dl, Ko, Vo, dst_token_offset=-1) == oracle.INVALID_ARG


def test_inject_rejects_damaged_cards():
    L, H, T, d = 1, 2, 16, 64
    Ks, Vs, lay = _cache(L, H, T, d, 68)
    _, card = oracle.card_create(lay, Ks, Vs, np.full(T, 4, np.uint8))
    Ko, Vo, dl = _cache(L, H, T, d, 69)
    for off, val in ((0, 0x00), (4, 9), (8, 3), (24, 128), (32, 16)):
        bad = card.copy()
        bad[off] = val
        assert oracle.card_inject(bad, dl, Ko, Vo) == oracle.BAD_CARD
    assert oracle.card_inject(card, dl, Ko, Vo, card_bytes=card.size - 1) == oracle.BAD_CARD
    assert oracle.card_inject(card, oracle.make_layout(L, H + 1, d, T), Ko, Vo) == oracle.BAD_CARD


def test_inject_rejects_damaged_stream_bases():
    """Per-head mode: a stream-base entry that is misaligned, points beyond the card, or sits so
    close to 2^64 that base + length wraps around to a small number, is refused."""
    L, H, T, d = 1, 2, 16, 64
    Ks, Vs, _ = _cache(L, H, T, d, 168)
    lay = oracle.make_layout(L, H, d, T, bits_mode=1)
    bits = np.concatenate([wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 169 + s) for s in range(L * H)])
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    hd = oracle.parse_header(card)
    Ko, Vo, _ = _cache(L, H, T, d, 170)
    dl = oracle.make_layout(L, H, d, T)
    assert oracle.card_inject(card, dl, Ko, Vo) == oracle.OK
    for value in (8, card.size, 2 ** 64 - 16 - hd["payload_off"], 2 ** 64 - 256, 2 ** 63):
        bad = card.copy()
        bad[hd["sbase_off"] + 8 * 2:hd["sbase_off"] + 8 * 3] = np.frombuffer(int(value).to_bytes(8, "little"), np.uint8)
        assert oracle.card_inject(bad, dl, Ko, Vo) == oracle.BAD_CARD
        assert oracle.card_attend(bad, oracle.make_layout(L, H, d, T), np.zeros((L, H, d), np.float16))[0] == oracle.BAD_CARD


def test_create_reports_bad_bits_and_short_buffer():
    L, H, T, d = 1, 1, 16, 64
    Ks, Vs, lay = _cache(L, H, T, d, 70)
    bits = np.full(T, 4, np.uint8)
    bits[7] = 5
    st, card = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.BAD_BITS and oracle.parse_header(card)["status"] == oracle.BAD_BITS
    good = np.full(T, 8, np.uint8)
    _, need = oracle.card_size(lay, good)
    st, card = oracle.card_create(lay, Ks, Vs, good, capacity=need - 16)
    assert st == oracle.BUFFER_TOO_SMALL
    assert oracle.parse_header(card)["status"] == oracle.BUFFER_TOO_SMALL
    st, _ = oracle.card_create(lay, Ks, Vs, good, capacity=300)
    assert st == oracle.BUFFER_TOO_SMALL


def test_per_head_bits_mode():
    """bits[L*H][T]: K and V of (layer, head) share a segment; stream bases are a running sum."""
    L, H, T, d = 2, 2, 24, 64
    Ks, Vs, _ = _cache(L, H, T, d, 71)
    lay = oracle.make_layout(L, H, d, T, bits_mode=1)
    bits = np.stack([wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 100 + i) for i in range(L * H)])
    st, card = oracle.card_create(lay, Ks, Vs, bits.reshape(-1))
    assert st == oracle.OK
    hd = oracle.parse_header(card)
    assert hd["bits_mode"] == 1 and hd["stream_bytes"] == 0 and hd["sbase_off"] > 0
    assert hd["total_bytes"] == card.size == oracle.card_size(lay, bits.reshape(-1))[1]
    sbase = card[hd["sbase_off"]:hd["sbase_off"] + 8 * (2 * L * H + 1)].view("<u8")
    pos = 0
    for l in range(L):
        for kv, arr in enumerate((Ks[l], Vs[l])):
            for h in range(H):
                s = (l * 2 + kv) * H + h
                enc = oracle.encode_stream(arr[h], bits[l * H + h])
                assert sbase[s] == pos
                b0 = hd["payload_off"] + pos
                assert np.array_equal(card[b0:b0 + enc.size], enc)
                pos += enc.size
    assert sbase[2 * L * H] == pos == card.size - hd["payload_off"]
    Ko, Vo, dl = _cache(L, H, T, d, 72)
    assert oracle.card_inject(card, dl, Ko, Vo) == oracle.OK
    for l in range(L):
        for h in range(H):
            want = oracle.decode_stream(oracle.encode_stream(Vs[l][h], bits[l * H + h]), bits[l * H + h], d)
            assert np.array_equal(Vo[l][h].view(np.uint16), want.view(np.uint16))


def test_card_is_position_independent():
    """All offsets are relative to the blob start: a copy at another address injects identically."""
    L, H, T, d = 1, 2, 20, 64
    Ks, Vs, lay = _cache(L, H, T, d, 73)
    _, card = oracle.card_create(lay, Ks, Vs, wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 3))
    moved = np.concatenate([np.zeros(48, np.uint8), card])[48:]
    Ka, Va, dl = _cache(L, H, T, d, 74)
    Kb, Vb, _ = _cache(L, H, T, d, 75)
    assert oracle.card_inject(card, dl, Ka, Va) == oracle.OK
    assert oracle.card_inject(moved, dl, Kb, Vb) == oracle.OK
    assert np.array_equal(Ka[0].view(np.uint16), Kb[0].view(np.uint16))


def test_tiny_config_card():
    """Config 1 (1 layer, 2 heads, d 64, 128 tokens, uniform 4-bit) end to end on the CPU."""
    w = wl.WORKLOADS[1]
    (_, K, V), = list(wl.kv_layers(w))
    bits = wl.bits_for(w)
    lay = oracle.make_layout(1, 2, 64, 128)
    st, card = oracle.card_create(lay, [K], [V], bits)
    assert st == oracle.OK
    assert card.size == 256 + 256 + 768 + 24576
    Ko, Vo = np.zeros_like(K), np.zeros_like(V)
    assert oracle.card_inject(card, lay, [Ko], [Vo]) == oracle.OK
    err = np.abs(Ko.astype(np.float32) - K.astype(np.float32)).max()
    assert 0 < err < 0.5


def test_card_of_appended_tokens_equals_slices_of_the_whole_card():
    """Records do not depend on a token's position: a card made from rows [t0, t0 + n) of a cache
    holds, stream by stream, bytes [off[t0], off[t0 + n)) of the whole cache's card, and injecting
    it at t0 rebuilds the same rows (incremental handoff: only what a hop appended)."""
    L, H, T, d, t0 = 2, 2, 90, 64, 53
    Ks, Vs, lay = _cache(L, H, T, d, 91)
    bits = np.random.default_rng(92).choice(np.array([2, 4, 8, 16], np.uint8), size=T)
    st, whole = oracle.card_create(lay, Ks, Vs, bits)
    assert st == oracle.OK
    n = T - t0
    part_lay = oracle.make_layout(L, H, d, n, head_stride=lay.head_stride, token_stride=lay.token_stride)
    st, part = oracle.card_create(part_lay, [k[:, t0:] for k in Ks], [v[:, t0:] for v in Vs], bits[t0:])
    assert st == oracle.OK
    hw, hp = oracle.parse_header(whole), oracle.parse_header(part)
    _, off, _ = oracle.scan_offsets(d, bits)
    assert hp["n_tokens"] == n and hp["stream_bytes"] == int(off[T] - off[t0])
    for s in range(2 * L * H):
        a = hw["payload_off"] + s * hw["stream_bytes"]
        b = hp["payload_off"] + s * hp["stream_bytes"]
        assert np.array_equal(part[b:b + hp["stream_bytes"]], whole[a + int(off[t0]):a + int(off[T])])
    Kw = [np.zeros((H, T, d), np.float16) for _ in range(L)]
    Vw = [np.zeros((H, T, d), np.float16) for _ in range(L)]
    assert oracle.card_inject(whole, lay, Kw, Vw) == oracle.OK
    Kp = [np.full((H, T, d), 9.0, np.float16) for _ in range(L)]
    Vp = [np.full((H, T, d), 9.0, np.float16) for _ in range(L)]
    assert oracle.card_inject(part, part_lay, Kp, Vp, dst_token_offset=t0) == oracle.OK
    for l in range(L):
        assert np.array_equal(Kp[l][:, t0:].view(np.uint16), Kw[l][:, t0:].view(np.uint16))
        assert np.array_equal(Vp[l][:, t0:].view(np.uint16), Vw[l][:, t0:].view(np.uint16))
        assert np.all(Kp[l][:, :t0] == 9.0) and np.all(Vp[l][:, :t0] == 9.0)
