"""Compact-metadata cards (FP16 scale rounded up + FP16 zero, 4 bytes per group): CUDA path
against the CPU oracle, through the C-ABI, on a B200.

Same bar as for the fp32-metadata format: the card (header, tables, payload, padding) is bit-exact
and nothing is written behind it; injected FP16 keys and values are within one FP16 unit in the
last place of the oracle's (observed: zero); attention from the card is within the tolerance
derived in test_gpu_attend.py.
"""
import numpy as np
import pytest

import oracle
import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from paper_2605_03884_b200 import workloads as wl
from golden_io import read_fixture
from rank_rule import by_library_sort
from gpu_utils import PAD, POISON, gpu_create, gpu_inject, max_ulp, padded_cache, to_cuda

pytestmark = pytest.mark.gpu

MAX_ULP = 1
META = 4


@pytest.fixture(scope="module", autouse=True)
def _library():
    qbuild.build()
    q.load_library()


def _olay(L, H, d, T, mode=0, meta_bytes=META, **strides):
    return oracle.make_layout(L, H, d, T, bits_mode=mode, meta_bytes=meta_bytes, **strides)


def _glay(L, H, d, T, mode=0, meta_bytes=META, **strides):
    return q.make_layout(L, H, d, T, bits_mode=mode, meta_bytes=meta_bytes, **strides)


def _check_card(Ks, Vs, bits, L, H, d, T, mode=0, strides=None, scratch=True):
    strides = strides or {}
    st_o, want = oracle.card_create(_olay(L, H, d, T, mode, **strides), Ks, Vs, bits, model_id=3, sender_id=9)
    assert st_o == oracle.OK
    st, hdr, whole, _ = gpu_create(q, _glay(L, H, d, T, mode, **strides), Ks, Vs, bits,
                                   meta=q.CardMeta(3, 9, 0), scratch=scratch)
    assert st == q.binding.OK
    assert hdr.meta_bytes_per_group == META and hdr.total_bytes == want.size
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


def test_record_sizes_through_the_library():
    fx = read_fixture("card_sizes.txt")
    for d, b, n in fx["crec"]:
        assert q.record_bytes(int(d), int(b), META) == int(n)
    assert q.record_bytes(64, 4, META) == 0 and q.record_bytes(192, 4, META) == 0
    assert q.record_bytes(128, 4, 2) == 0
    assert q.record_bytes(128, 4, 0) == q.record_bytes(128, 4, 8) == 96


def test_worked_examples_on_the_gpu():
    """The hand-worked groups D and E as one-token cards."""
    for name in ("compact_example_d_2bit.txt", "compact_example_e_4bit.txt"):
        fx = read_fixture(name)
        b = int(fx["bits"][0][0])
        x = np.array([float(v) for v in fx["x"][0]], dtype=np.float16)
        K = np.tile(x, 4).reshape(1, 1, 128)
        st, hdr, whole, _ = gpu_create(q, _glay(1, 1, 128, 1), [K], [K.copy()], np.array([b], np.uint8))
        assert st == q.binding.OK
        rec = whole[hdr.payload_off:hdr.payload_off + q.record_bytes(128, b, META)]
        assert rec[:16].view("<u2").tolist() == [int(fx["scale_bits"][0][0], 16), int(fx["zero_bits"][0][0], 16)] * 4
        assert rec[16:].tolist() == [int(v, 16) for v in fx["packed_hex"][0]] * 4
        stat, Kg, _ = gpu_inject(q, whole[:hdr.total_bytes], _glay(1, 1, 128, 1), [np.zeros_like(K)], [np.zeros_like(K)])
        assert stat == 0
        assert Kg[0].astype(np.float64).reshape(-1).tolist() == [float(v) for v in fx["dequant"][0]] * 4


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("T", [1, 31, 64, 65, 333])
def test_mixed_bits_ragged_tiles(d, T):
    L, H = 2, 3
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=2000 + d + T)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=d * 11 + T)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_uniform_bits(b):
    L, H, d, T = 1, 2, 128, 200
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=50 + b)
    card = _check_card(Ks, Vs, np.full(T, b, np.uint8), L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


@pytest.mark.parametrize("spread", [1e-3, 1.0, 300.0])
def test_value_scales(spread):
    """Small, ordinary and large magnitudes: the round-up of the scale crosses FP16 binades and,
    for the small ones, the subnormal range."""
    L, H, d, T = 1, 2, 128, 160
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=70, scale=spread)
    bits = wl.iid_bits(T, (0.35, 0.35, 0.25, 0.05), seed=71)
    card = _check_card(Ks, Vs, bits, L, H, d, T)
    assert _check_inject(card, L, H, d, T) == 0


def test_adversarial_values():
    """Constant groups, signed zeros, largest magnitudes, subnormals, huge dynamic range, ties."""
    L, H, d, T = 1, 1, 128, 96
    rng = np.random.default_rng(9)
    K = (rng.standard_normal((H, T, d), dtype=np.float32)).astype(np.float16)
    V = K.copy()
    K[0, 0] = 1.25
    K[0, 1] = 0.0
    K[0, 1, ::2] = -0.0
    K[0, 2, :32] = 0.0
    K[0, 2, 1:32:2] = -0.0
    K[0, 2, 5] = 3.0
    K[0, 3, ::2], K[0, 3, 1::2] = 65504.0, -65504.0          # largest range: scale 131008/3 rounded up
    K[0, 4] = (np.arange(d, dtype=np.uint16) * 5).view(np.float16)   # subnormals
    K[0, 5] = (rng.standard_normal(d) * 1e-4).astype(np.float16)
    K[0, 6] = (rng.standard_normal(d) * 2e4).astype(np.float16)
    K[0, 7, :32] = np.arange(32) * 0.25 - 1.5
    K[0, 7, 31] = 6.0
    K[0, 8] = -np.abs(K[0, 8])
    K[0, 8, 3] = -0.0
    K[0, 9, :] = 6e-8
    K[0, 10, :64] = 1e-7
    K[0, 10, 64:] = 60000.0
    K[0, 11, :] = 0.0
    K[0, 11, 7] = np.float16(2.0 ** -24)                     # smallest range: scale 2^-24 at every width
    for bits in (np.full(T, 2, np.uint8), np.full(T, 4, np.uint8), np.full(T, 8, np.uint8),
                 wl.iid_bits(T, (0.3, 0.3, 0.3, 0.1), 4)):
        card = _check_card([K], [V], bits, L, H, d, T)
        assert _check_inject(card, L, H, d, T) == 0


def test_without_scratch_block_and_many_chunks():
    L, H, d, T = 4, 8, 128, 5000
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=4343)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), seed=98)
    for scratch in (True, False):
        card = _check_card(Ks, Vs, bits, L, H, d, T, scratch=scratch)
        assert _check_inject(card, L, H, d, T, scratch=scratch) == 0


def test_strided_source_padded_destination_and_per_head_bits():
    L, H, d, T = 2, 2, 128, 100
    Ks, Vs, strides = padded_cache(L, H, T, d, seed=21, t_cap=120, token_stride=136)
    bits = np.stack([wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 400 + i) for i in range(L * H)]).reshape(-1)
    card = _check_card(Ks, Vs, bits, L, H, d, T, mode=1, strides=strides)
    assert _check_inject(card, L, H, d, T, dst_strides=dict(token_stride=144), t_cap=160,
                         dst_token_offset=37) == 0


def test_shape_and_format_mismatches():
    """head_dim 64 / 192 cannot carry 4-byte metadata; a card is only read back with the format it
    was made with, in both directions, and nothing is written otherwise."""
    import torch
    for d in (64, 192):
        with pytest.raises(q.binding.QkvsError) as e:
            q.card_size(_glay(1, 1, d, 8), None)
        assert e.value.status == q.binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(q.binding.QkvsError) as e:
        q.card_size(_glay(1, 1, 128, 8, meta_bytes=2), None)
    assert e.value.status == q.binding.ERR_INVALID_ARG
    L, H, d, T = 1, 2, 128, 40
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=5)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=6)
    st4, c4 = oracle.card_create(_olay(L, H, d, T), Ks, Vs, bits)
    st8, c8 = oracle.card_create(_olay(L, H, d, T, meta_bytes=8), Ks, Vs, bits)
    assert st4 == st8 == oracle.OK
    blank = [np.full((H, T, d), -3.0, np.float16)]
    for card, meta in ((c4, 8), (c8, 4)):
        st, Kg, Vg = gpu_inject(q, card, _glay(L, H, d, T, meta_bytes=meta), blank, blank)
        assert st == q.binding.ERR_BAD_CARD and np.all(Kg[0] == -3.0) and np.all(Vg[0] == -3.0)
    torch.cuda.synchronize()


def test_attention_from_a_compact_card():
    import torch
    L, H, d, nq = 2, 2, 128, 8
    for T in (1, 17, 256, 1000):
        Ks, Vs, _ = padded_cache(L, H, T, d, seed=600 + T)
        bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=T + 1)
        olay = _olay(L, H, d, T)
        st, card = oracle.card_create(olay, Ks, Vs, bits)
        assert st == oracle.OK
        qh = wl.random_fp16((L, nq, d), 950 + T)
        st, want = oracle.card_attend(card, olay, qh)
        assert st == oracle.OK
        lay = _glay(L, H, d, T)
        out = torch.full(qh.shape, 7.0, dtype=torch.float32, device="cuda")
        scratch = torch.full((q.attend_scratch_size(lay, nq),), 0x5A, dtype=torch.uint8, device="cuda")
        q.card_attend(torch.from_numpy(card).cuda(), lay, torch.from_numpy(qh).cuda(), out, scratch)
        torch.cuda.synchronize()
        assert int(scratch[:4].view(torch.int32).item()) == 0
        got = out.cpu().numpy()
        Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
        assert oracle.card_inject(card, olay, Kr, Vr) == oracle.OK
        for l in range(L):
            for j in range(nq):
                vmax = float(np.abs(Vr[l][j // (nq // H)].astype(np.float64)).max())
                assert float(np.abs(got[l, j] - want[l, j]).max()) <= 2.0 ** -9 * vmax + 1e-6
        # the other format's kernel refuses this card
        lay8 = _glay(L, H, d, T, meta_bytes=8)
        q.card_attend(torch.from_numpy(card).cuda(), lay8, torch.from_numpy(qh).cuda(), out, scratch)
        torch.cuda.synchronize()
        assert int(scratch[:4].view(torch.int32).item()) == q.binding.ERR_BAD_CARD
        assert not out.any()


def test_llama_8k_adaptive_full_size():
    """The 8K adaptive workload (all four widths) at full size with compact metadata: whole card
    bit-exact, whole injected cache equal to the oracle's, with the launch shape the benchmark uses."""
    import torch
    w = wl.WORKLOADS[4]
    Ks, Vs = [], []
    for _, k, v in wl.kv_layers(w):
        Ks.append(k)
        Vs.append(v)
    bits = wl.bits_for(w, rank_rule=by_library_sort)
    L, H, d, T = w.n_layers, w.n_kv_heads, w.head_dim, w.n_tokens
    st_o, want = oracle.card_create(_olay(L, H, d, T), Ks, Vs, bits)
    assert st_o == oracle.OK
    fx = read_fixture("card_sizes.txt")
    assert want.size == q.card_prefix_size(_glay(L, H, d, T)) + int(fx["cpayload"][1][-1])
    Kd, Vd = to_cuda(Ks), to_cuda(Vs)
    size = q.card_size(_glay(L, H, d, T), bits)
    assert size == want.size
    buf = torch.full((size + PAD,), POISON, dtype=torch.uint8, device="cuda")
    ws = q.new_workspace()
    q.card_create(_glay(L, H, d, T), Kd, Vd, torch.from_numpy(bits).cuda(), buf, card_capacity=size, workspace=ws)
    st, hdr = q.card_info(buf)
    assert st == 0 and hdr.total_bytes == size
    got = buf.cpu().numpy()
    assert np.array_equal(got[:size], want)
    assert np.all(got[size:] == POISON)
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
    assert worst == 0


def test_per_head_bits_attention_and_injection_without_a_scratch_block():
    """The remaining combinations of the compact format: per-(layer, head) bit-widths under
    attention, and the entry point that keeps its work counters in the library's own memory."""
    import torch
    L, H, d, T, nq = 2, 2, 128, 300, 8
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=910)
    bits = np.stack([wl.iid_bits(T, (0.25, 0.25, 0.25, 0.25), 920 + i) for i in range(L * H)]).reshape(-1)
    olay, glay = _olay(L, H, d, T, mode=1), _glay(L, H, d, T, mode=1)
    st, card = oracle.card_create(olay, Ks, Vs, bits)
    assert st == oracle.OK
    qh = wl.random_fp16((L, nq, d), 930)
    st, want = oracle.card_attend(card, olay, qh)
    assert st == oracle.OK
    card_d = torch.from_numpy(card).cuda()
    out = torch.full(qh.shape, 7.0, dtype=torch.float32, device="cuda")
    scratch = torch.full((q.attend_scratch_size(glay, nq),), 0x5A, dtype=torch.uint8, device="cuda")
    q.card_attend(card_d, glay, torch.from_numpy(qh).cuda(), out, scratch)
    torch.cuda.synchronize()
    assert int(scratch[:4].view(torch.int32).item()) == 0
    Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, olay, Kr, Vr) == oracle.OK
    got = out.cpu().numpy()
    for l in range(L):
        for j in range(nq):
            vmax = float(np.abs(Vr[l][j // (nq // H)].astype(np.float64)).max())
            assert float(np.abs(got[l, j] - want[l, j]).max()) <= 2.0 ** -9 * vmax + 1e-6
    # injection through the entry point without a scratch block: the oracle's values
    Ko = [torch.full((H, T, d), -3.0, dtype=torch.float16, device="cuda") for _ in range(L)]
    Vo = [torch.full((H, T, d), -5.0, dtype=torch.float16, device="cuda") for _ in range(L)]
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    assert q.card_inject_noalloc(card_d, glay, Ko, Vo, status_dev=status) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for l in range(L):
        assert max_ulp(Ko[l].cpu().numpy(), Kr[l]) == 0 and max_ulp(Vo[l].cpu().numpy(), Vr[l]) == 0
