"""Parity of the CUDA path with the CPU oracle, through the C-ABI, on a B200.

Cards (header, tables, payload) must be bit-exact, byte for byte, including padding; injected
FP16 keys and values may differ from the oracle's by at most one FP16 unit in the last place
(the tests additionally record that the observed difference is zero).
"""
import numpy as np
import pytest

import oracle
import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from paper_2605_03884_b200 import workloads as wl
from gpu_utils import PAD, POISON, gpu_create, gpu_inject, max_ulp, padded_cache, to_cuda
from rank_rule import by_library_sort

pytestmark = pytest.mark.gpu

MAX_ULP = 1  # FP16 keys/values: at most 1 ulp from the oracle


@pytest.fixture(scope="module", autouse=True)
def _library():
    qbuild.build()
    q.load_library()


def _olay(L, H, d, T, mode=0, **strides):
    return oracle.make_layout(L, H, d, T, bits_mode=mode, **strides)


def _glay(L, H, d, T, mode=0, **strides):
    return q.make_layout(L, H, d, T, bits_mode=mode, **strides)


def _check_card(Ks, Vs, bits, L, H, d, T, mode=0, strides=None, meta=(0, 0, 0), scratch=True):
    strides = strides or {}
    st_o, want = oracle.card_create(_olay(L, H, d, T, mode, **strides), Ks, Vs, bits,
                                    model_id=meta[0], sender_id=meta[1], position_offset=meta[2])
    assert st_o == oracle.OK
    st, hdr, whole, cap = gpu_create(q, _glay(L, H, d, T, mode, **strides), Ks, Vs, bits,
                                     meta=q.CardMeta(*meta), scratch=scratch)
    assert st == q.binding.OK
    assert hdr.total_bytes == want.size
    got = whole[:want.size]
    if not np.array_equal(got, want):
        bad = np.flatnonzero(got != want)
        raise AssertionError(f"card differs at {bad.size} bytes, first at {bad[0]} "
                             f"(payload_off {hdr.payload_off}): got {got[bad[0]]:#x} want {want[bad[0]]:#x}")
    assert np.all(whole[want.size:] == POISON), "bytes behind the card were written"
    return want


def _check_inject(card, L, H, d, T, dst_strides=None, t_cap=None, dst_token_offset=0, scratch=True):
    dst_strides = dst_strides or {}
    t_cap = T if t_cap is None else t_cap
    ts = dst_strides.get("token_stride", d)
    Ko = [np.full((H, t_cap, ts), -3.0, np.float16) for _ in range(L)]
    Vo = [np.full((H, t_cap, ts), -5.0, np.float16) for _ in range(L)]
    Kw, Vw = [a.copy() for a in Ko], [a.copy() for a in Vo]
    lay_kw = dict(head_stride=t_cap * ts, token_stride=ts)
    assert oracle.card_inject(card, _olay(L, H, d, T, **lay_kw), Kw, Vw, dst_token_offset) == oracle.OK
    st, Kg, Vg = gpu_inject(q, card, _glay(L, H, d, T, **lay_kw), Ko, Vo, dst_token_offset, scratch=scratch)
    assert st == (0 if scratch else None)
    worst = 0
    for l in range(L):
        for g, w in ((Kg[l], Kw[l]), (Vg[l], Vw[l])):
            worst = max(worst, max_ulp(g, w))
    assert worst <= MAX_ULP
    return worst


# ----------------------------------------------------------------------------- configs 1, 2

def test_config1_tiny_uniform4():
    w = wl.WORKLOADS[1]
    (_, K, V), = list(wl.kv_layers(w))
    card = _check_card([K], [V], wl.bits_for(w), 1, 2, 64, 128)
    assert _check_inject(card, 1, 2, 64, 128) == 0


@pytest.mark.parametrize("d", [64, 128, 192, 256])
@pytest.mark.parametrize("T", [1, 31, 64, 65, 333])
def test_mixed_bits_ragged_tiles(d, T):
    """Several tiles plus a ragged tail, all four bit-widths alternating token by token."""
    L, H = 2, 3
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=1000 + d + T)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=d * 7 + T)
    card = _check_card(Ks, Vs, bits, L, H, d, T, meta=(0xABCDEF0123456789, 77, -12))
    assert _check_inject(card, L, H, d, T) == 0


@pytest.mark.parametrize("d,T", [(64, 700), (128, 2100), (192, 333), (256, 517)])
def test_without_scratch_block(d, T):
    """No scratch block: the work is split in advance instead of drawn from a counter; the
    results are the same bytes."""
    L, H = 3, 4
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=77 + d)
    bits = wl.iid_bits(T, (0.35, 0.35, 0.2, 0.1), seed=d + T)
    card = _check_card(Ks, Vs, bits, L, H, d, T, scratch=False)
    assert _check_inject(card, L, H, d, T, scratch=False) == 0


def test_many_chunks_per_warp():
    """More chunks than the grid has warps, so that every warp draws several from the counter
    (and, without a scratch block, strides through several)."""
    L, H, d, T = 4, 8, 128, 9000
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=4242)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), seed=99)
    for scratch in (True, False):
        card = _check_card(Ks, Vs, bits, L, H, d, T, scratch=scratch)
        assert _check_inject(card, L, H, d, T, scratch=scratch) == 0


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_uniform_bits(b):
    L, H, d, T = 1, 2, 128, 200
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=b)
    card = _check_card(Ks, Vs, np.full(T, b, np.uint8), L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


def test_alternating_bits_every_token():
    L, H, d, T = 1, 2, 128, 256
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=5)
    bits = np.tile(np.array([2, 16, 4, 8], np.uint8), T // 4)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


def test_adversarial_values():
    """Constant groups, signed zeros, largest magnitudes, subnormals, huge dynamic range, ties."""
    L, H, d, T = 1, 1, 128, 96
    rng = np.random.default_rng(9)
    K = (rng.standard_normal((H, T, d), dtype=np.float32)).astype(np.float16)
    V = K.copy()
    K[0, 0] = 1.25                                  # constant row
    K[0, 1] = 0.0
    K[0, 1, ::2] = -0.0                             # only zeros, mixed signs
    K[0, 2, :32] = 0.0
    K[0, 2, 1:32:2] = -0.0
    K[0, 2, 5] = 3.0                                # zero minimum stored as +0
    K[0, 3, ::2], K[0, 3, 1::2] = 65504.0, -65504.0
    K[0, 4] = (np.arange(d, dtype=np.uint16) * 5).view(np.float16)       # subnormals
    K[0, 5] = (rng.standard_normal(d) * 1e-4).astype(np.float16)
    K[0, 6] = (rng.standard_normal(d) * 2e4).astype(np.float16)
    K[0, 7, :32] = np.arange(32) * 0.25 - 1.5       # exact ties at 4 bits
    K[0, 7, 31] = 6.0
    K[0, 8] = -np.abs(K[0, 8])                      # all negative
    K[0, 8, 3] = -0.0
    K[0, 9, :] = 6e-8                               # constant subnormal
    K[0, 10, :64] = 1e-7
    K[0, 10, 64:] = 60000.0
    for bits in (np.full(T, 2, np.uint8), np.full(T, 4, np.uint8), np.full(T, 8, np.uint8),
                 wl.iid_bits(T, (0.3, 0.3, 0.3, 0.1), 4)):
        card = _check_card([K], [V], bits, L, H, d, T)
        assert _check_inject(card, L, H, d, T) == 0


def test_fp16_tokens_keep_every_bit_pattern():
    """All 65536 FP16 patterns (NaN payloads, infinities, -0, subnormals) survive create+inject."""
    L, H, d, T = 1, 1, 128, 512
    K = np.arange(65536, dtype=np.uint32).astype(np.uint16).view(np.float16).reshape(1, T, d)
    V = K[:, ::-1].copy()
    bits = np.full(T, 16, np.uint8)
    card = _check_card([K], [V], bits, L, H, d, T)
    st, Kg, Vg = gpu_inject(q, card, _glay(L, H, d, T), [np.zeros_like(K)], [np.zeros_like(V)])
    assert st == 0
    assert np.array_equal(Kg[0].view(np.uint16), K.view(np.uint16))
    assert np.array_equal(Vg[0].view(np.uint16), V.view(np.uint16))


def test_strided_source_and_padded_destination():
    L, H, d, T = 2, 2, 64, 100
    Ks, Vs, strides = padded_cache(L, H, T, d, seed=21, t_cap=120, token_stride=72)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 22)
    card = _check_card(Ks, Vs, bits, L, H, d, T, strides=strides)
    # destination with a different row pitch, more capacity, and an offset; untouched bytes stay
    assert _check_inject(card, L, H, d, T, dst_strides=dict(token_stride=80), t_cap=160,
                         dst_token_offset=37) == 0


def test_per_head_bits_mode():
    L, H, d, T = 2, 2, 128, 150
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=31)
    bits = np.stack([wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 300 + i) for i in range(L * H)]).reshape(-1)
    card = _check_card(Ks, Vs, bits, L, H, d, T, mode=1)
    assert _check_inject(card, L, H, d, T) == 0


def test_long_context_with_a_ragged_end():
    """131 109 tokens of one (layer, head): far beyond the benchmark's lengths, offsets past 2^24,
    a last sub-tile of five rows; whole card and whole cache compared."""
    L, H, d, T = 1, 1, 128, 131072 + 37
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=43)
    bits = wl.iid_bits(T, (0.3, 0.4, 0.2, 0.1), 44)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


def test_many_layers_span_several_launches():
    """More layers than one launch's pointer block carries."""
    L, H, d, T = 70, 1, 64, 20
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=41)
    bits = wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 42)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


def test_card_survives_a_copy_to_another_address():
    """The blob is position independent: device -> host -> another device address -> inject."""
    import torch
    L, H, d, T = 1, 2, 128, 70
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=51)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 52)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    big = torch.zeros(card.size + 4096, dtype=torch.uint8, device="cuda")
    big[1024:1024 + card.size] = torch.from_numpy(card).cuda()
    Kd, Vd = to_cuda([np.zeros((H, T, d), np.float16)]), to_cuda([np.zeros((H, T, d), np.float16)])
    q.card_inject(big[1024:1024 + card.size], _glay(L, H, d, T), Kd, Vd, card_bytes=card.size)
    Kw, Vw = [np.zeros((H, T, d), np.float16)], [np.zeros((H, T, d), np.float16)]
    assert oracle.card_inject(card, _olay(L, H, d, T), Kw, Vw) == oracle.OK
    assert np.array_equal(Kd[0].cpu().numpy().view(np.uint16), Kw[0].view(np.uint16))
    assert np.array_equal(Vd[0].cpu().numpy().view(np.uint16), Vw[0].view(np.uint16))


def test_card_of_appended_tokens_only():
    """A hop that appended tokens hands on only those: the card is made from row t0 of the cache
    on (pointers to that row, n_tokens = what was appended) and injected at t0.  Bit-exact against
    the oracle given the same rows; the destination's earlier rows stay untouched."""
    import torch
    L, H, d, T, t0 = 2, 3, 128, 333, 200
    Ks, Vs, strides = padded_cache(L, H, T, d, seed=55, t_cap=400, token_stride=136)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=56)
    n = T - t0
    olay, glay = _olay(L, H, d, n, **strides), _glay(L, H, d, n, **strides)
    st_o, want = oracle.card_create(olay, [k[:, t0:] for k in Ks], [v[:, t0:] for v in Vs], bits[t0:])
    assert st_o == oracle.OK
    Kd, Vd = to_cuda(Ks), to_cuda(Vs)
    buf = torch.full((want.size + PAD,), POISON, dtype=torch.uint8, device="cuda")
    q.card_create(glay, Kd, Vd, torch.from_numpy(bits[t0:]).cuda(), buf, card_capacity=want.size,
                  workspace=q.new_workspace(), src_token_offset=t0)
    st, hdr = q.card_info(buf)
    got = buf.cpu().numpy()
    assert st == 0 and hdr.n_tokens == n
    assert np.array_equal(got[:want.size], want) and np.all(got[want.size:] == POISON)
    Ko = [np.full_like(k, -3.0) for k in Ks]
    Vo = [np.full_like(v, -5.0) for v in Vs]
    Kw, Vw = [a.copy() for a in Ko], [a.copy() for a in Vo]
    assert oracle.card_inject(want, olay, Kw, Vw, t0) == oracle.OK
    stat, Kg, Vg = gpu_inject(q, want, glay, Ko, Vo, dst_token_offset=t0)
    assert stat == 0
    for l in range(L):
        assert np.array_equal(Kg[l].view(np.uint16), Kw[l].view(np.uint16))
        assert np.array_equal(Vg[l].view(np.uint16), Vw[l].view(np.uint16))
        assert np.all(Kg[l][:, :t0] == -3.0) and np.all(Vg[l][:, :t0] == -5.0)


def test_empty_card():
    L, H, d, T = 1, 2, 64, 0
    Ks = [np.zeros((H, 1, d), np.float16)]
    st, hdr, whole, cap = gpu_create(q, _glay(L, H, d, T, head_stride=d), Ks, Ks, np.zeros(0, np.uint8))
    st_o, want = oracle.card_create(_olay(L, H, d, T, head_stride=d), Ks, Ks, np.zeros(0, np.uint8))
    assert st == 0 and st_o == 0 and hdr.total_bytes == want.size
    assert np.array_equal(whole[:want.size], want)


# ----------------------------------------------------------------------------- device-detected errors

def test_bad_bits_reported_in_header_and_no_payload():
    L, H, d, T = 1, 2, 128, 100
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=61)
    bits = np.full(T, 4, np.uint8)
    bits[63] = 5
    st, hdr, whole, cap = gpu_create(q, _glay(L, H, d, T), Ks, Vs, bits)
    assert st == q.binding.ERR_BAD_BITS and hdr.status == q.binding.ERR_BAD_BITS
    assert np.all(whole[hdr.payload_off:] == POISON)
    st_o, _ = oracle.card_create(_olay(L, H, d, T), Ks, Vs, bits)
    assert st_o == oracle.BAD_BITS


def test_short_buffer_reported_and_nothing_written_beyond_it():
    L, H, d, T = 1, 2, 128, 100
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=62)
    bits = np.full(T, 8, np.uint8)
    need = q.card_size(_glay(L, H, d, T), bits)
    st, hdr, whole, cap = gpu_create(q, _glay(L, H, d, T), Ks, Vs, bits, capacity=need - 16)
    assert st == q.binding.ERR_BUFFER_TOO_SMALL
    assert np.all(whole[hdr.payload_off:] == POISON)
    st, hdr, whole, cap = gpu_create(q, _glay(L, H, d, T), Ks, Vs, bits, capacity=need)
    assert st == 0 and np.all(whole[need:] == POISON)


def test_inject_refuses_damaged_cards_without_writing():
    L, H, d, T = 1, 2, 128, 100
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=63)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 64)
    _, card = oracle.card_create(_olay(L, H, d, T), Ks, Vs, bits)
    hd = oracle.parse_header(card)

    def damaged(off, val):
        c = card.copy()
        c[off] = val
        return c

    cases = [damaged(0, 0), damaged(4, 7), damaged(8, 3), damaged(24, 64), damaged(28, 99),
             damaged(hd["bits_off"] + 10, 3),                    # bit-width not in the set
             damaged(hd["offs_off"] + 4 * 20, card[hd["offs_off"] + 4 * 20] ^ 0x10)]  # offset off
    swapped = card.copy()
    swapped[hd["bits_off"] + 5] = 16 if bits[5] != 16 else 2     # valid width, wrong record size
    cases.append(swapped)
    for c in cases:
        Ko = [np.full((H, T, d), -3.0, np.float16)]
        Vo = [np.full((H, T, d), -5.0, np.float16)]
        st, Kg, Vg = gpu_inject(q, c, _glay(L, H, d, T), Ko, Vo)
        assert st == q.binding.ERR_BAD_CARD
    # header-level damage leaves the destination untouched
    for c in cases[:5]:
        st, Kg, Vg = gpu_inject(q, c, _glay(L, H, d, T), [np.full((H, T, d), -3.0, np.float16)],
                                [np.full((H, T, d), -5.0, np.float16)])
        assert np.all(Kg[0] == -3.0) and np.all(Vg[0] == -5.0)
    # a card cut short is refused on the device (total_bytes beyond what the caller says is valid)
    st, Kg, Vg = gpu_inject(q, card, _glay(L, H, d, T), [np.full((H, T, d), -3.0, np.float16)],
                            [np.full((H, T, d), -5.0, np.float16)], card_bytes=card.size - 16)
    assert st == q.binding.ERR_BAD_CARD and np.all(Kg[0] == -3.0)
    # shape mismatch
    st, Kg, Vg = gpu_inject(q, card, _glay(L, H, d, T - 1), [np.full((H, T, d), -3.0, np.float16)],
                            [np.full((H, T, d), -5.0, np.float16)])
    assert st == q.binding.ERR_BAD_CARD and np.all(Kg[0] == -3.0)


def test_inject_refuses_damaged_stream_bases():
    """Per-head mode: a stream-base entry that is misaligned, beyond the card, or so close to 2^64
    that base + length would wrap around.  The card sits in the interior of a larger device tensor,
    so every address a wrong sum could form still lies in mapped memory.  The damaged stream's rows
    stay untouched, the others are injected, and the status word says BAD_CARD."""
    import torch
    L, H, d, T = 1, 2, 128, 100
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=163)
    bits = np.concatenate([wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), 164 + s) for s in range(L * H)])
    _, card = oracle.card_create(_olay(L, H, d, T, mode=1), Ks, Vs, bits)
    hd = oracle.parse_header(card)
    Kw, Vw = [np.zeros((H, T, d), np.float16)], [np.zeros((H, T, d), np.float16)]
    assert oracle.card_inject(card, _olay(L, H, d, T), Kw, Vw) == oracle.OK
    margin = 1 << 20
    victim = 2                                  # stream (layer 0, V, head 0)
    for value in (8, card.size, card.size + 4096, 2 ** 64 - 16 - hd["payload_off"], 2 ** 64 - 4096, 2 ** 63):
        bad = card.copy()
        bad[hd["sbase_off"] + 8 * victim:hd["sbase_off"] + 8 * (victim + 1)] = np.frombuffer(int(value).to_bytes(8, "little"), np.uint8)
        assert oracle.card_inject(bad, _olay(L, H, d, T), [k.copy() for k in Kw], [v.copy() for v in Vw]) == oracle.BAD_CARD
        big = torch.full((2 * margin + card.size,), POISON, dtype=torch.uint8, device="cuda")
        big[margin:margin + card.size] = torch.from_numpy(bad).cuda()
        inner = big[margin:margin + card.size]
        Kd = to_cuda([np.full((H, T, d), -3.0, np.float16)])
        Vd = to_cuda([np.full((H, T, d), -5.0, np.float16)])
        ws = q.new_workspace()
        q.card_inject(inner, _glay(L, H, d, T), Kd, Vd, card_bytes=card.size, workspace=ws)
        torch.cuda.synchronize()
        assert int(ws[0].item()) == q.binding.ERR_BAD_CARD
        Kg, Vg = Kd[0].cpu().numpy(), Vd[0].cpu().numpy()
        assert np.all(Vg[0] == -5.0), "rows of the damaged stream were written"
        assert np.array_equal(Kg.view(np.uint16), Kw[0].view(np.uint16))
        assert np.array_equal(Vg[1].view(np.uint16), Vw[0][1].view(np.uint16))


def test_worked_examples_on_the_gpu():
    """The stored hand-worked groups (exact ties at 4, 2 and 8 bits; the group with an inexact
    scale at all three widths) as one-token cards: scale, zero and packed codes as stored."""
    from golden_io import read_fixture
    cases = []
    for name in ("worked_example_a_4bit.txt", "worked_example_b_2bit.txt", "worked_example_c_8bit.txt"):
        fx = read_fixture(name)
        x = np.array([float(v) for v in fx["x"][0]], dtype=np.float16)
        cases.append((int(fx["bits"][0][0]), x, int(fx["scale_bits"][0][0], 16), int(fx["zero_bits"][0][0], 16),
                      [int(v, 16) for v in fx["packed_hex"][0]], [float(v) for v in fx["dequant"][0]]))
    fx = read_fixture("worked_example_f_inexact.txt")
    xf = np.array([int(v) for v in fx["x_bits"][0]], dtype=np.uint16).view(np.float16)
    for (b, scale_hex, _), packed in zip(fx["case"], fx["packed_hex"]):
        cases.append((int(b), xf, int(scale_hex, 16), int(fx["zero_bits"][0][0], 16), [int(v, 16) for v in packed], None))
    for b, x, scale_bits, zero_bits, packed, dequant in cases:
        K = np.tile(x, 4).reshape(1, 1, 128)
        st, hdr, whole, _ = gpu_create(q, _glay(1, 1, 128, 1), [K], [K.copy()], np.array([b], np.uint8))
        assert st == q.binding.OK
        rec = whole[hdr.payload_off:hdr.payload_off + q.record_bytes(128, b)]
        assert rec[:32].view("<u4").tolist() == [scale_bits, zero_bits] * 4
        assert rec[32:].tolist() == packed * 4
        stat, Kg, _ = gpu_inject(q, whole[:hdr.total_bytes], _glay(1, 1, 128, 1), [np.zeros_like(K)], [np.zeros_like(K)])
        assert stat == 0
        if dequant is not None:
            assert Kg[0].astype(np.float64).reshape(-1).tolist() == dequant * 4


def test_card_sent_to_a_buffer_of_its_own_injects_identically():
    """qkvs_card_send on the one GPU at hand: the copy holds the same bytes, and injecting from it
    (a different address, other bytes around it) rebuilds the same cache as the oracle.  Unknown
    devices and a device that is neither end of the copy are refused."""
    import torch
    L, H, d, T = 2, 2, 128, 333
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=81)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), 82)
    want = _check_card(Ks, Vs, bits, L, H, d, T)
    src = torch.from_numpy(want).cuda()
    dst = torch.full((want.size + 4096,), POISON, dtype=torch.uint8, device="cuda")
    q.card_send(src, dst[2048:], card_bytes=want.size)
    torch.cuda.synchronize()
    got = dst.cpu().numpy()
    assert np.array_equal(got[2048:2048 + want.size], want)
    assert np.all(got[:2048] == POISON) and np.all(got[2048 + want.size:] == POISON)
    assert _check_inject(got[2048:2048 + want.size], L, H, d, T) == 0
    n = torch.cuda.device_count()
    lib = q.load_library()
    st = lib.qkvs_card_send(src.data_ptr(), want.size, 0, dst.data_ptr(), dst.numel(), n, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = q.card_send(src, dst[:want.size - 16], card_bytes=want.size, check=False)
    assert st == q.binding.ERR_BUFFER_TOO_SMALL


def test_a_wait_that_nothing_completes_gives_up_and_reports_it():
    """The kernels' only waits are bounded; this runs one on a barrier that never completes, with a
    limit of five milliseconds: the kernel returns, the status word says TIMEOUT, the wait lasted
    about as long as asked, and the path works afterwards."""
    import torch
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    q.selftest_bounded_wait(5000, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == q.binding.ERR_TIMEOUT
    assert 5_000_000 <= int(waited.item()) < 500_000_000
    L, H, d, T = 1, 2, 128, 50
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=71)
    card = _check_card(Ks, Vs, np.full(T, 4, np.uint8), L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


# ----------------------------------------------------------------------------- full-size configs

def _full_config(number):
    w = wl.WORKLOADS[number]
    Ks, Vs = [], []
    for _, k, v in wl.kv_layers(w):
        Ks.append(k)
        Vs.append(v)
    return w, Ks, Vs


def _full_parity(w, Ks, Vs, bits):
    """Whole card bit-exact and whole injected cache within MAX_ULP at the benchmark's size,
    through the same entry points and launch configuration bench.py times."""
    import torch
    L, H, d, T = w.n_layers, w.n_kv_heads, w.head_dim, w.n_tokens
    st_o, want = oracle.card_create(_olay(L, H, d, T), Ks, Vs, bits)
    assert st_o == oracle.OK
    Kd, Vd = to_cuda(Ks), to_cuda(Vs)
    bits_d = torch.from_numpy(bits).cuda()
    size = q.card_size(_glay(L, H, d, T), bits)
    assert size == want.size
    buf = torch.full((size + PAD,), POISON, dtype=torch.uint8, device="cuda")
    ws = q.new_workspace()
    q.card_create(_glay(L, H, d, T), Kd, Vd, bits_d, buf, card_capacity=size, workspace=ws)
    st, hdr = q.card_info(buf)
    assert st == 0 and hdr.total_bytes == size
    got = buf.cpu().numpy()
    assert np.array_equal(got[:size], want)
    assert np.all(got[size:] == POISON)
    # inject on the GPU, oracle inject on the CPU
    Ko = [torch.zeros_like(k) for k in Kd]
    Vo = [torch.zeros_like(v) for v in Vd]
    q.card_inject(buf, _glay(L, H, d, T), Ko, Vo, card_bytes=size, workspace=ws)
    assert int(ws[0].item()) == 0
    Kw = [np.zeros_like(k) for k in Ks]
    Vw = [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(want, _olay(L, H, d, T), Kw, Vw) == oracle.OK
    worst = 0
    for l in range(L):
        worst = max(worst, max_ulp(Ko[l].cpu().numpy(), Kw[l]), max_ulp(Vo[l].cpu().numpy(), Vw[l]))
    assert worst <= MAX_ULP
    # FP16 tokens are exact copies of the input
    m = bits == 16
    if m.any():
        assert np.array_equal(Ko[0].cpu().numpy()[:, m].view(np.uint16), Ks[0][:, m].view(np.uint16))
    return worst, Ko, Vo


def test_config2_llama_1k_mixed_full():
    w, Ks, Vs = _full_config(2)
    worst, _, _ = _full_parity(w, Ks, Vs, wl.bits_for(w))
    assert worst == 0


def test_config3_llama_8k_uniform4_full():
    w, Ks, Vs = _full_config(3)
    worst, _, _ = _full_parity(w, Ks, Vs, wl.bits_for(w))
    assert worst == 0


def test_config4_llama_8k_adaptive_full():
    w, Ks, Vs = _full_config(4)
    bits = wl.bits_for(w, rank_rule=by_library_sort)
    assert abs(float(bits.astype(np.float64).mean()) - 4.4) < 0.01
    worst, _, _ = _full_parity(w, Ks, Vs, bits)
    assert worst == 0


def test_config5_chain_of_four_hops_full():
    """Each hop re-quantises the previous hop's GPU output; the oracle is fed the same bytes, so
    every hop's card must be bit-exact.  The pure-oracle chain must end at the same cache."""
    w, Ks, Vs = _full_config(5)
    L = w.n_layers
    K0 = [k.astype(np.float32) for k in Ks[:2]]
    Kc, Vc = Ks, Vs
    errs = []
    for hop in range(w.hops):
        bits = wl.bits_for(w, hop)
        worst, Ko, Vo = _full_parity(w, Kc, Vc, bits)
        assert worst == 0
        Kc = [k.cpu().numpy() for k in Ko]
        Vc = [v.cpu().numpy() for v in Vo]
        del Ko, Vo
        e = np.concatenate([(Kc[l].astype(np.float32) - K0[l]).reshape(-1) for l in range(2)])
        errs.append(float(np.sqrt(np.mean(e.astype(np.float64) ** 2))))
    assert all(np.isfinite(errs)) and errs[0] > 0
    # error accumulates but stays bounded by a few first-hop errors (soft check)
    assert errs[-1] < 4 * errs[0] + 1e-3


def test_division_shortcuts_equal_ieee_division_exhaustively():
    """Both division shortcuts of the quantiser agree with the IEEE quotient on every reachable
    operand (all binary32 ranges from 2^-24 to 131008, qmax in {3, 15, 255})."""
    import torch
    counts = torch.full((2,), -1, dtype=torch.int64, device="cuda")
    q.selftest_division(counts)
    torch.cuda.synchronize()
    assert counts.tolist() == [0, 0]
