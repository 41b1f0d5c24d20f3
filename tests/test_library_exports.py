"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed),
and its host-only entry points agree with the closed forms."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from golden_io import read_fixture

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    qbuild.build()
    return q.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "qkvshare.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qkvs_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(names) == set(q.binding.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_host_only_sizes(lib):
    fx = read_fixture("card_sizes.txt")
    for d, b, n in fx["rec"]:
        assert q.record_bytes(int(d), int(b)) == int(n)
    assert q.record_bytes(128, 3) == 0 and q.record_bytes(96, 4) == 0
    a = lambda x: (x + 255) // 256 * 256
    for L, H, d, T, c16, c8, c4, c2, payload in fx["payload"]:
        L, H, d, T = int(L), int(H), int(d), int(T)
        bits = np.concatenate([np.full(int(c16), 16), np.full(int(c8), 8), np.full(int(c4), 4),
                               np.full(int(c2), 2)]).astype(np.uint8)
        lay = q.make_layout(L, H, d, T)
        assert q.card_size(lay, bits) == 256 + a(T) + a(4 * (T + 1)) + int(payload)
        assert q.card_prefix_size(lay) == 256 + a(T) + a(4 * (T + 1))
    lay = q.make_layout(2, 2, 64, 10)
    assert q.card_size(lay, None) == q.card_size(lay, np.full(10, 16, np.uint8))
    with pytest.raises(q.QkvsError) as e:
        q.card_size(lay, np.array([4] * 9 + [5], np.uint8))
    assert e.value.status == q.binding.ERR_BAD_BITS
    with pytest.raises(q.QkvsError) as e:
        q.card_size(q.make_layout(1, 1, 96, 4), None)
    assert e.value.status == q.binding.ERR_UNSUPPORTED_SHAPE
    # per-head bits: K and V of a (layer, head) share one segment
    lay1 = q.make_layout(2, 3, 64, 5, bits_mode=1)
    bits = np.tile(np.array([2, 4, 8, 16, 4], np.uint8), 6)
    per_seg = 32 + 48 + 80 + 128 + 48
    assert q.card_size(lay1, bits) == 256 + a(30) + a(4 * 6 * 6) + a(8 * 13) + 12 * per_seg
    # compact metadata: four bytes per group, head_dim a multiple of 128
    for d, b, n in fx["crec"]:
        assert q.record_bytes(int(d), int(b), 4) == int(n)
    assert q.record_bytes(64, 4, 4) == 0 and q.record_bytes(128, 4, 3) == 0
    assert q.record_bytes(128, 4, 0) == q.record_bytes(128, 4, 8)
    for L, H, d, T, c16, c8, c4, c2, payload in fx["cpayload"]:
        L, H, d, T = int(L), int(H), int(d), int(T)
        bits = np.concatenate([np.full(int(c16), 16), np.full(int(c8), 8), np.full(int(c4), 4),
                               np.full(int(c2), 2)]).astype(np.uint8)
        assert q.card_size(q.make_layout(L, H, d, T, meta_bytes=4), bits) == 256 + a(T) + a(4 * (T + 1)) + int(payload)
    with pytest.raises(q.QkvsError) as e:
        q.card_size(q.make_layout(1, 1, 64, 4, meta_bytes=4), None)
    assert e.value.status == q.binding.ERR_UNSUPPORTED_SHAPE
    with pytest.raises(q.QkvsError) as e:
        q.card_size(q.make_layout(1, 1, 128, 4, meta_bytes=16), None)
    assert e.value.status == q.binding.ERR_INVALID_ARG


def test_status_strings_and_version(lib):
    assert q.version() >= 100
    seen = {q.status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_host_side_argument_checks_need_no_gpu(lib):
    """Errors knowable on the host come back before any CUDA call."""
    lay = q.make_layout(1, 1, 64, 4)
    null = C.c_void_p(0)
    arr = (C.c_void_p * 1)(0)
    st = lib.qkvs_card_create(C.byref(lay), arr, arr, null, None, null, 0, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    bad = q.make_layout(1, 1, 64, 4, token_stride=60)
    ptrs = (C.c_void_p * 1)(256)
    st = lib.qkvs_card_create(C.byref(bad), ptrs, ptrs, C.c_void_p(256), None, C.c_void_p(256), 1 << 20, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    mis = (C.c_void_p * 1)(264)
    st = lib.qkvs_card_create(C.byref(lay), mis, ptrs, C.c_void_p(256), None, C.c_void_p(256), 1 << 20, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_card_create(C.byref(lay), ptrs, ptrs, C.c_void_p(256), None, C.c_void_p(256), 100, None, None)
    assert st == q.binding.ERR_BUFFER_TOO_SMALL
    st = lib.qkvs_card_inject(C.c_void_p(256), 100, C.byref(lay), ptrs, ptrs, 0, None, None)
    assert st == q.binding.ERR_BAD_CARD
    st = lib.qkvs_card_inject(C.c_void_p(256), 4096, C.byref(lay), ptrs, ptrs, -1, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    # a scratch block has to be 16-byte aligned
    st = lib.qkvs_card_inject(C.c_void_p(256), 4096, C.byref(lay), ptrs, ptrs, 0, C.c_void_p(264), None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_card_create(C.byref(lay), ptrs, ptrs, C.c_void_p(256), None, C.c_void_p(256), 1 << 20,
                              C.c_void_p(264), None)
    assert st == q.binding.ERR_INVALID_ARG
    # row and stride arithmetic that would not fit 64 bits is refused, not wrapped
    st = lib.qkvs_card_inject(C.c_void_p(256), 4096, C.byref(lay), ptrs, ptrs, 2 ** 62, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    huge = q.make_layout(1, 4, 64, 4, head_stride=2 ** 61, token_stride=64)
    st = lib.qkvs_card_inject(C.c_void_p(256), 4096, C.byref(huge), ptrs, ptrs, 0, None, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_selftest_bounded_wait(0, C.c_void_p(256), None, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_selftest_bounded_wait(2_000_000, C.c_void_p(256), None, None)
    assert st == q.binding.ERR_INVALID_ARG
    # handing a card to another GPU: everything knowable without a device is checked first
    st = lib.qkvs_card_send(None, 4096, 0, C.c_void_p(256), 4096, 0, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_card_send(C.c_void_p(256), 4096, 0, C.c_void_p(264), 4096, 0, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_card_send(C.c_void_p(256), 4096, -1, C.c_void_p(512), 4096, 0, None)
    assert st == q.binding.ERR_INVALID_ARG
    st = lib.qkvs_card_send(C.c_void_p(256), 100, 0, C.c_void_p(512), 4096, 0, None)
    assert st == q.binding.ERR_BAD_CARD
    st = lib.qkvs_card_send(C.c_void_p(256), 4096, 0, C.c_void_p(512), 4095, 0, None)
    assert st == q.binding.ERR_BUFFER_TOO_SMALL


def test_controller_argument_checks_need_no_gpu(lib):
    p = C.c_void_p(256)
    f = lib.qkvs_bits_from_features
    assert f(p, -1, 46, p, p, None, None) == q.binding.ERR_INVALID_ARG
    assert f(p, 10, 0, p, p, None, None) == q.binding.ERR_INVALID_ARG
    assert f(p, 10, 129, p, p, None, None) == q.binding.ERR_UNSUPPORTED_SHAPE
    assert f(None, 10, 46, p, p, None, None) == q.binding.ERR_INVALID_ARG
    assert f(C.c_void_p(258), 10, 46, p, p, None, None) == q.binding.ERR_INVALID_ARG
    assert f(p, 10, 46, p, p, C.c_void_p(258), None) == q.binding.ERR_INVALID_ARG
    assert f(None, 0, 46, None, None, None, None) == q.binding.OK   # no tokens: nothing to do
