"""Groups of 64 and 128 channels (one scale / zero pair per wider group): CUDA path against the
oracle through the C-ABI.  Cards bit-exact, injected values within one FP16 unit (observed: 0)."""
import numpy as np
import pytest

import oracle
import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from paper_2605_03884_b200 import workloads as wl
from gpu_utils import POISON, gpu_create, gpu_inject, max_ulp, padded_cache

pytestmark = pytest.mark.gpu

COMBOS = [(d, g, m) for d in (128, 256) for g in (64, 128) for m in (8, 4)]


@pytest.fixture(scope="module", autouse=True)
def _library():
    qbuild.build()
    q.load_library()


def _round_trip(Ks, Vs, bits, L, H, d, T, group, meta, mode=0, strides=None):
    strides = strides or {}
    olay = oracle.make_layout(L, H, d, T, bits_mode=mode, meta_bytes=meta, group_size=group, **strides)
    glay = q.make_layout(L, H, d, T, bits_mode=mode, meta_bytes=meta, group_size=group, **strides)
    st_o, want = oracle.card_create(olay, Ks, Vs, bits)
    assert st_o == oracle.OK
    st, hdr, whole, cap = gpu_create(q, glay, Ks, Vs, bits)
    assert st == q.binding.OK and hdr.total_bytes == want.size and hdr.group_size == group
    got = whole[:want.size]
    if not np.array_equal(got, want):
        bad = np.flatnonzero(got != want)
        raise AssertionError(f"card differs at {bad.size} bytes, first at {bad[0]} (payload_off {hdr.payload_off})")
    assert np.all(whole[want.size:] == POISON)
    dl_o = oracle.make_layout(L, H, d, T, meta_bytes=meta, group_size=group)
    dl_g = q.make_layout(L, H, d, T, meta_bytes=meta, group_size=group)
    Kw = [np.full((H, T, d), -3.0, np.float16) for _ in range(L)]
    Vw = [np.full((H, T, d), -5.0, np.float16) for _ in range(L)]
    assert oracle.card_inject(want, dl_o, Kw, Vw) == oracle.OK
    stat, Kg, Vg = gpu_inject(q, want, dl_g, [np.full((H, T, d), -3.0, np.float16) for _ in range(L)],
                              [np.full((H, T, d), -5.0, np.float16) for _ in range(L)])
    assert stat == 0
    worst = max(max(max_ulp(Kg[l], Kw[l]), max_ulp(Vg[l], Vw[l])) for l in range(L))
    assert worst <= 1
    return want, worst


@pytest.mark.parametrize("d,group,meta", COMBOS)
@pytest.mark.parametrize("T", [1, 31, 333])
def test_mixed_bits_ragged_tiles(d, group, meta, T):
    L, H = 2, 3
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=3000 + d + group + meta + T)
    bits = wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=d + group + T)
    _, worst = _round_trip(Ks, Vs, bits, L, H, d, T, group, meta)
    assert worst == 0


@pytest.mark.parametrize("d,group,meta", COMBOS)
@pytest.mark.parametrize("b", [2, 4, 8, 16])
def test_uniform_bits(d, group, meta, b):
    L, H, T = 1, 2, 200
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=b + group)
    _, worst = _round_trip(Ks, Vs, np.full(T, b, np.uint8), L, H, d, T, group, meta)
    assert worst == 0


def test_outlier_channels_constant_groups_and_per_head_bits():
    """Keys with outlier channels (what stretches a wide group's range), constant groups, signed
    zeros, and the per-(layer, head) bit-width mode."""
    L, H, d, T = 2, 2, 128, 150
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=77)
    for k in Ks:
        k[:, :, 5] *= np.float16(10.0)
        k[:, 10:20, 64:128] = np.float16(0.75)       # constant groups of 64
        k[:, 20:30, :] = np.float16(-0.0)
    bits = np.concatenate([wl.iid_bits(T, (0.3, 0.3, 0.3, 0.1), 78 + s) for s in range(L * H)])
    for group in (64, 128):
        _round_trip(Ks, Vs, bits, L, H, d, T, group, 8, mode=1)


def test_sizes_padding_and_mismatch_are_refused():
    import torch
    lay = q.make_layout(2, 2, 128, 10, group_size=64)
    bits = np.full(10, 4, np.uint8)
    assert q.card_size(lay, bits) == q.card_prefix_size(lay) + 2 * 2 * 2 * 10 * 80
    assert q.card_size(q.make_layout(1, 1, 256, 10, group_size=128, meta_bytes=4), bits) - q.card_prefix_size(q.make_layout(1, 1, 256, 10, group_size=128)) == 2 * 10 * 144
    for bad in (q.make_layout(1, 1, 64, 4, group_size=64), q.make_layout(1, 1, 192, 4, group_size=64), q.make_layout(1, 1, 128, 4, group_size=48)):
        with pytest.raises(q.QkvsError) as e:
            q.card_size(bad, None)
        assert e.value.status == q.binding.ERR_UNSUPPORTED_SHAPE
    # a card is read back with the group size it was made with
    L, H, d, T = 1, 2, 128, 40
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=5)
    _, card = oracle.card_create(oracle.make_layout(L, H, d, T, group_size=64), Ks, Vs, np.full(T, 4, np.uint8))
    for other in (32, 128):
        stat, Kg, _ = gpu_inject(q, card, q.make_layout(L, H, d, T, group_size=other), [np.full((H, T, d), -3.0, np.float16)],
                                 [np.full((H, T, d), -5.0, np.float16)])
        assert stat == q.binding.ERR_BAD_CARD and np.all(Kg[0] == -3.0)


def _attend(card_np, lay, qh):
    import torch
    card = torch.from_numpy(np.ascontiguousarray(card_np)).cuda()
    out = torch.full(qh.shape, 7.0, dtype=torch.float32, device="cuda")
    scratch = torch.full((q.attend_scratch_size(lay, qh.shape[1]),), 0x5A, dtype=torch.uint8, device="cuda")
    q.card_attend(card, lay, torch.from_numpy(qh).cuda(), out, scratch)
    torch.cuda.synchronize()
    return int(scratch[:4].view(torch.int32).item()), out.cpu().numpy()


@pytest.mark.parametrize("group,meta", [(64, 8), (64, 4), (128, 8), (128, 4)])
@pytest.mark.parametrize("T,uniform", [(1, 0), (100, 0), (530, 0), (1000, 4), (300, 2), (300, 8)])
def test_attention_from_a_wide_group_card(group, meta, T, uniform):
    """Attention straight from the card reads wide groups too (head_dim 128): against the oracle's
    attention over the values the records stand for, tolerance as for groups of 32
    (2^-9 of the head's largest reconstructed value: the weights are rounded to FP16)."""
    L, H, d, nq = 2, 2, 128, 8
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=40 + T)
    bits = np.full(T, uniform, np.uint8) if uniform else wl.iid_bits(T, (0.3, 0.3, 0.2, 0.2), seed=T)
    olay = oracle.make_layout(L, H, d, T, meta_bytes=meta, group_size=group)
    st, card = oracle.card_create(olay, Ks, Vs, bits)
    assert st == oracle.OK
    qh = wl.random_fp16((L, nq, d), 77 + T)
    st, want = oracle.card_attend(card, olay, qh)
    assert st == oracle.OK
    status, got = _attend(card, q.make_layout(L, H, d, T, meta_bytes=meta, group_size=group), qh)
    assert status == 0
    Kr, Vr = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(card, olay, Kr, Vr) == oracle.OK
    for l in range(L):
        for j in range(nq):
            vmax = float(np.abs(Vr[l][j // (nq // H)][:T, :d].astype(np.float64)).max())
            assert float(np.abs(got[l, j] - want[l, j]).max()) <= 2.0 ** -9 * vmax + 1e-6, (l, j)


def test_attention_refuses_a_card_of_another_group_size():
    L, H, d, T = 1, 2, 128, 40
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=6)
    _, card = oracle.card_create(oracle.make_layout(L, H, d, T, group_size=64), Ks, Vs, np.full(T, 4, np.uint8))
    qh = wl.random_fp16((L, 4, d), 7)
    for other in (32, 128):
        status, got = _attend(card, q.make_layout(L, H, d, T, group_size=other), qh)
        assert status == q.binding.ERR_BAD_CARD and np.all(got == 0.0)


def test_full_size_llama_8k_adaptive_groups_of_64():
    """The 8K adaptive workload with one fp32 pair per 64 channels, whole card and whole cache."""
    import torch
    from rank_rule import by_library_sort
    from gpu_utils import to_cuda
    w = wl.WORKLOADS[4]
    Ks, Vs = [], []
    for _, k, v in wl.kv_layers(w):
        Ks.append(k)
        Vs.append(v)
    bits = wl.bits_for(w, rank_rule=by_library_sort)
    L, H, d, T = w.n_layers, w.n_kv_heads, w.head_dim, w.n_tokens
    olay = oracle.make_layout(L, H, d, T, group_size=64)
    glay = q.make_layout(L, H, d, T, group_size=64)
    st_o, want = oracle.card_create(olay, Ks, Vs, bits)
    assert st_o == oracle.OK
    Kd, Vd = to_cuda(Ks), to_cuda(Vs)
    size = q.card_size(glay, bits)
    assert size == want.size
    buf = torch.full((size + 512,), POISON, dtype=torch.uint8, device="cuda")
    ws = q.new_workspace()
    q.card_create(glay, Kd, Vd, torch.from_numpy(bits).cuda(), buf, card_capacity=size, workspace=ws)
    st, hdr = q.card_info(buf)
    assert st == 0 and hdr.total_bytes == size
    got = buf.cpu().numpy()
    assert np.array_equal(got[:size], want) and np.all(got[size:] == POISON)
    Ko = [torch.zeros_like(k) for k in Kd]
    Vo = [torch.zeros_like(v) for v in Vd]
    q.card_inject(buf, glay, Ko, Vo, card_bytes=size, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws[0].item()) == 0
    Kw, Vw = [np.zeros_like(k) for k in Ks], [np.zeros_like(v) for v in Vs]
    assert oracle.card_inject(want, olay, Kw, Vw) == oracle.OK
    for l in range(L):
        assert np.array_equal(Ko[l].cpu().numpy().view(np.uint16), Kw[l].view(np.uint16))
        assert np.array_equal(Vo[l].cpu().numpy().view(np.uint16), Vw[l].view(np.uint16))
