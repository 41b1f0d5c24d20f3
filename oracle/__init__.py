"""Python face of the CPU oracle (test infrastructure, not a product path).

Compiles `qkvs_oracle.c` with gcc on first use and calls it through ctypes with numpy
arrays.  Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package; the CUDA library never does, and nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qkvs_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libqkvs_oracle.so")

OK, INVALID_ARG, UNSUPPORTED_SHAPE, BAD_BITS, BUFFER_TOO_SMALL, BAD_CARD = range(6)


class Layout(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_tokens", C.c_int32), ("group_size", C.c_int32), ("bits_mode", C.c_int32),
                ("head_stride", C.c_int64), ("token_stride", C.c_int64),
                ("meta_bytes", C.c_int32), ("reserved_", C.c_int32)]


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, no fused multiply-add, OpenMP over streams)."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_LIB_PATH)
             or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
    if force or stale:
        tmp = _LIB_PATH + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


_lib = None


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        u8p, u16p, u32p = C.POINTER(C.c_uint8), C.POINTER(C.c_uint16), C.POINTER(C.c_uint32)
        l.orc_half_to_float.restype = C.c_float
        l.orc_half_to_float.argtypes = [C.c_uint16]
        l.orc_float_to_half.restype = C.c_uint16
        l.orc_float_to_half.argtypes = [C.c_float]
        l.orc_record_bytes.restype = C.c_int64
        l.orc_record_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        l.orc_record_bytes_g.restype = C.c_int64
        l.orc_record_bytes_g.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
        l.orc_scan_offsets_g.restype = C.c_int
        l.orc_scan_offsets_g.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_void_p, C.POINTER(C.c_uint64)]
        l.orc_quantize_span.restype = None
        l.orc_quantize_span.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_void_p]
        l.orc_quantize_span_compact.restype = None
        l.orc_quantize_span_compact.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16), C.c_void_p]
        l.orc_dequantize_span.restype = None
        l.orc_dequantize_span.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_float, C.c_void_p]
        l.orc_encode_stream_g.restype = None
        l.orc_encode_stream_g.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        l.orc_decode_stream_g.restype = None
        l.orc_decode_stream_g.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64]
        l.orc_scan_offsets.restype = C.c_int
        l.orc_scan_offsets.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_void_p, C.POINTER(C.c_uint64)]
        l.orc_card_size.restype = C.c_int
        l.orc_card_size.argtypes = [C.POINTER(Layout), C.c_void_p, C.POINTER(C.c_uint64)]
        l.orc_quantize_group.restype = None
        l.orc_quantize_group.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_void_p]
        l.orc_quantize_group_compact.restype = None
        l.orc_quantize_group_compact.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_uint16), C.POINTER(C.c_uint16), C.c_void_p]
        l.orc_float_to_half_up.restype = C.c_uint16
        l.orc_float_to_half_up.argtypes = [C.c_float]
        l.orc_dequantize_group.restype = None
        l.orc_dequantize_group.argtypes = [C.c_void_p, C.c_float, C.c_float, C.c_void_p]
        l.orc_pack_codes.restype = None
        l.orc_pack_codes.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        l.orc_unpack_codes.restype = None
        l.orc_unpack_codes.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        l.orc_encode_stream.restype = None
        l.orc_encode_stream.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        l.orc_decode_stream.restype = None
        l.orc_decode_stream.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_int64]
        l.orc_write_prefix.restype = C.c_int
        l.orc_write_prefix.argtypes = [C.POINTER(Layout), C.c_void_p, C.c_uint64, C.c_uint64, C.c_int64, C.c_void_p, C.c_uint64]
        l.orc_card_create_range.restype = C.c_int
        l.orc_card_create_range.argtypes = [C.POINTER(Layout), C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                            C.c_uint64, C.c_int64, C.c_void_p, C.c_uint64, C.c_int64, C.c_int64]
        l.orc_card_inject.restype = C.c_int
        l.orc_card_inject.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(Layout), C.c_void_p, C.c_void_p, C.c_int64]
        l.orc_bits_from_scores.restype = C.c_int
        l.orc_bits_from_scores.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_void_p]
        l.orc_bits_from_scores_budget.restype = C.c_int
        l.orc_bits_from_scores_budget.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_uint64, C.c_void_p, C.c_void_p]
        l.orc_combine_scores.restype = C.c_int
        l.orc_combine_scores.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_int64, C.c_void_p]
        l.orc_bits_from_features.restype = C.c_int
        l.orc_bits_from_features.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        l.orc_card_attend.restype = C.c_int
        l.orc_card_attend.argtypes = [C.c_void_p, C.c_uint64, C.POINTER(Layout), C.c_int, C.c_void_p, C.c_double, C.c_void_p]
        l.orc_card_attend_injected.restype = C.c_int
        l.orc_card_attend_injected.argtypes = l.orc_card_attend.argtypes
        l.orc_num_threads.restype = C.c_int
        l.orc_set_num_threads.argtypes = [C.c_int]
        _lib = l
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def make_layout(n_layers, n_kv_heads, head_dim, n_tokens, bits_mode=0, head_stride=None,
                token_stride=None, meta_bytes=8, group_size=32) -> Layout:
    ts = head_dim if token_stride is None else token_stride
    hs = n_tokens * ts if head_stride is None else head_stride
    return Layout(n_layers, n_kv_heads, head_dim, n_tokens, group_size, bits_mode, hs, ts, meta_bytes, 0)


def half_to_float(h: int) -> float:
    return float(lib().orc_half_to_float(int(h)))


def float_to_half(f: float) -> int:
    return int(lib().orc_float_to_half(C.c_float(f)))


def record_bytes(head_dim: int, b: int, meta_bytes: int = 8, group_size: int = 32) -> int:
    return int(lib().orc_record_bytes_g(head_dim, b, meta_bytes, group_size))


def scan_offsets(head_dim: int, bits: np.ndarray, meta_bytes: int = 8, group_size: int = 32) -> Tuple[int, np.ndarray, int]:
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    off = np.zeros(bits.size + 1, dtype=np.uint32)
    sb = C.c_uint64(0)
    st = lib().orc_scan_offsets_g(head_dim, meta_bytes, group_size, _ptr(bits), bits.size, _ptr(off), C.byref(sb))
    return st, off, int(sb.value)


def quantize_span(x: np.ndarray, b: int, compact: bool = False):
    """One group of n = x.size (32, 64 or 128) FP16 values -> (scale, zero, codes[n]); with
    compact=True scale and zero come back as FP16 values."""
    x = np.ascontiguousarray(x).view(np.uint16)
    n = x.size
    assert n in (32, 64, 128)
    q = np.zeros(n, dtype=np.uint8)
    if compact:
        s, z = C.c_uint16(0), C.c_uint16(0)
        lib().orc_quantize_span_compact(_ptr(x), n, b, C.byref(s), C.byref(z), _ptr(q))
        return (np.array([s.value], dtype=np.uint16).view(np.float16)[0],
                np.array([z.value], dtype=np.uint16).view(np.float16)[0], q)
    s, z = C.c_float(0), C.c_float(0)
    lib().orc_quantize_span(_ptr(x), n, b, C.byref(s), C.byref(z), _ptr(q))
    return np.float32(s.value), np.float32(z.value), q


def dequantize_span(q: np.ndarray, scale, zero) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    out = np.zeros(q.size, dtype=np.uint16)
    lib().orc_dequantize_span(_ptr(q), q.size, C.c_float(scale), C.c_float(zero), _ptr(out))
    return out.view(np.float16)


def card_size(layout: Layout, bits: Optional[np.ndarray]) -> Tuple[int, int]:
    out = C.c_uint64(0)
    if bits is not None:
        bits = np.ascontiguousarray(bits, dtype=np.uint8)
    st = lib().orc_card_size(C.byref(layout), None if bits is None else _ptr(bits), C.byref(out))
    return st, int(out.value)


def quantize_group(x: np.ndarray, b: int) -> Tuple[float, float, np.ndarray]:
    """x: 32 FP16 values (float16 or uint16 bit patterns) -> (scale, zero, codes[32])."""
    x = np.ascontiguousarray(x).view(np.uint16)
    assert x.size == 32
    q = np.zeros(32, dtype=np.uint8)
    s, z = C.c_float(0), C.c_float(0)
    lib().orc_quantize_group(_ptr(x), b, C.byref(s), C.byref(z), _ptr(q))
    return np.float32(s.value), np.float32(z.value), q


def quantize_group_compact(x: np.ndarray, b: int) -> Tuple[np.float16, np.float16, np.ndarray]:
    """x: 32 FP16 values -> (scale, zero, codes[32]) with scale and zero as FP16 values."""
    x = np.ascontiguousarray(x).view(np.uint16)
    assert x.size == 32
    q = np.zeros(32, dtype=np.uint8)
    s, z = C.c_uint16(0), C.c_uint16(0)
    lib().orc_quantize_group_compact(_ptr(x), b, C.byref(s), C.byref(z), _ptr(q))
    return (np.array([s.value], dtype=np.uint16).view(np.float16)[0],
            np.array([z.value], dtype=np.uint16).view(np.float16)[0], q)


def float_to_half_up(f: float) -> int:
    return int(lib().orc_float_to_half_up(C.c_float(f)))


def dequantize_group(q: np.ndarray, scale, zero) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    out = np.zeros(32, dtype=np.uint16)
    lib().orc_dequantize_group(_ptr(q), C.c_float(scale), C.c_float(zero), _ptr(out))
    return out.view(np.float16)


def pack_codes(q: np.ndarray, b: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    out = np.zeros(q.size * b // 8, dtype=np.uint8)
    lib().orc_pack_codes(_ptr(q), q.size, b, _ptr(out))
    return out


def unpack_codes(packed: np.ndarray, n: int, b: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    q = np.zeros(n, dtype=np.uint8)
    lib().orc_unpack_codes(_ptr(packed), n, b, _ptr(q))
    return q


def encode_stream(x: np.ndarray, bits: np.ndarray, meta_bytes: int = 8, group_size: int = 32) -> np.ndarray:
    """One [T, d] FP16 matrix + bits[T] -> the stream's payload bytes."""
    x = np.ascontiguousarray(x).view(np.uint16)
    t, d = x.shape
    st, off, _ = scan_offsets(d, bits, meta_bytes, group_size)
    if st:
        raise ValueError(f"bad bits (status {st})")
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.zeros(int(off[-1]), dtype=np.uint8)
    lib().orc_encode_stream_g(_ptr(x), d, t, d, meta_bytes, group_size, _ptr(bits), _ptr(off), _ptr(out))
    return out


def decode_stream(payload: np.ndarray, bits: np.ndarray, d: int, meta_bytes: int = 8, group_size: int = 32) -> np.ndarray:
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    st, off, _ = scan_offsets(d, bits, meta_bytes, group_size)
    if st:
        raise ValueError(f"bad bits (status {st})")
    assert payload.size == int(off[-1])
    x = np.zeros((bits.size, d), dtype=np.uint16)
    lib().orc_decode_stream_g(_ptr(payload), _ptr(bits), _ptr(off), bits.size, d, meta_bytes, group_size, _ptr(x), d)
    return x.view(np.float16)


def _ptr_array(arrs: Sequence[np.ndarray]):
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def write_prefix(layout: Layout, bits: np.ndarray, model_id=0, sender_id=0, position_offset=0,
                 capacity: Optional[int] = None) -> Tuple[int, np.ndarray]:
    """Header + bits + offsets (+ stream bases) only; returns (status, bytes)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    st, total = card_size(layout, bits)
    if st:
        st2, worst = card_size(layout, None)
        total = worst
    cap = total if capacity is None else capacity
    card = np.zeros(max(cap, 256), dtype=np.uint8)
    st = lib().orc_write_prefix(C.byref(layout), _ptr(bits), model_id, sender_id, position_offset,
                                _ptr(card), cap)
    return st, card


def card_create(layout: Layout, K_layers: List[np.ndarray], V_layers: List[np.ndarray],
                bits: np.ndarray, model_id=0, sender_id=0, position_offset=0,
                capacity: Optional[int] = None, streams: Optional[Tuple[int, int]] = None
                ) -> Tuple[int, np.ndarray]:
    """Whole card (or only the streams in `streams`) from per-layer FP16 arrays.

    K_layers[l] / V_layers[l] are arrays whose memory is addressed with the layout's strides
    (head_stride, token_stride, in elements) from their first element.
    """
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    st, total = card_size(layout, bits)
    if st:
        _, total = card_size(layout, None)
    cap = total if capacity is None else capacity
    card = np.zeros(max(cap, 256), dtype=np.uint8)
    S = 2 * layout.n_layers * layout.n_kv_heads
    s0, s1 = (0, S) if streams is None else streams
    kp, vp = _ptr_array(K_layers), _ptr_array(V_layers)
    st = lib().orc_card_create_range(C.byref(layout), kp, vp, _ptr(bits), model_id, sender_id,
                                     position_offset, _ptr(card), cap, s0, s1)
    return st, card


def card_create_into(layout: Layout, K_layers: List[np.ndarray], V_layers: List[np.ndarray],
                     bits: np.ndarray, card: np.ndarray, model_id=0, sender_id=0, position_offset=0) -> int:
    """The same call writing into a caller's buffer (uint8, at least card_size bytes): nothing is
    allocated, so a stopwatch around it times the oracle's own work."""
    assert card.dtype == np.uint8 and card.flags["C_CONTIGUOUS"] and bits.dtype == np.uint8
    S = 2 * layout.n_layers * layout.n_kv_heads
    kp, vp = _ptr_array(K_layers), _ptr_array(V_layers)
    return lib().orc_card_create_range(C.byref(layout), kp, vp, _ptr(bits), model_id, sender_id,
                                       position_offset, _ptr(card), card.size, 0, S)


def card_inject(card: np.ndarray, dst: Layout, K_out: List[np.ndarray], V_out: List[np.ndarray],
                dst_token_offset: int = 0, card_bytes: Optional[int] = None) -> int:
    card = np.ascontiguousarray(card, dtype=np.uint8)
    kp, vp = _ptr_array(K_out), _ptr_array(V_out)
    return lib().orc_card_inject(_ptr(card), card.size if card_bytes is None else card_bytes,
                                 C.byref(dst), kp, vp, dst_token_offset)


def card_attend(card: np.ndarray, layout: Layout, q: np.ndarray, softmax_scale: Optional[float] = None,
                injected: bool = False) -> Tuple[int, np.ndarray]:
    """Decode-step attention from the card.  q: FP16 [n_layers, n_q_heads, head_dim]; returns
    (status, float64 [n_layers, n_q_heads, head_dim]).  injected=False attends to the values the
    records stand for (unrounded); injected=True to the FP16 cache injection would rebuild."""
    card = np.ascontiguousarray(card, dtype=np.uint8)
    q = np.ascontiguousarray(q, dtype=np.float16)
    assert q.ndim == 3 and q.shape[0] == layout.n_layers and q.shape[2] == layout.head_dim
    scale = 1.0 / float(np.sqrt(layout.head_dim)) if softmax_scale is None else float(softmax_scale)
    out = np.zeros(q.shape, dtype=np.float64)
    fn = lib().orc_card_attend_injected if injected else lib().orc_card_attend
    st = fn(_ptr(card), card.size, C.byref(layout), q.shape[1], _ptr(q), scale, _ptr(out))
    return st, out


def bits_from_scores(scores: np.ndarray, n_fp16: int, n_8bit: int, n_4bit: int) -> Tuple[int, np.ndarray]:
    """Per-token bit-widths from float32 scores [T] by rank (see orc_bits_from_scores)."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    bits = np.zeros(scores.size, dtype=np.uint8)
    st = lib().orc_bits_from_scores(_ptr(scores), scores.size, n_fp16, n_8bit, n_4bit, _ptr(bits))
    return st, bits


DEFAULT_UPGRADE_WEIGHTS = (2.0 ** -9, 2.0 ** -14, 2.0 ** -23)


def bits_from_scores_budget(scores: np.ndarray, head_dim: int, budget_bytes: int, weights=DEFAULT_UPGRADE_WEIGHTS,
                            meta_bytes: int = 8) -> Tuple[int, np.ndarray]:
    """Per-token bit-widths from float32 scores [T] under a byte budget per stream (see
    orc_bits_from_scores_budget)."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    w = np.ascontiguousarray(weights, dtype=np.float32)
    assert w.size == 3
    bits = np.zeros(scores.size, dtype=np.uint8)
    st = lib().orc_bits_from_scores_budget(_ptr(scores), scores.size, head_dim, meta_bytes, int(budget_bytes), _ptr(w), _ptr(bits))
    return st, bits


def combine_scores(importance: np.ndarray, transfer: np.ndarray, alpha: float) -> Tuple[int, np.ndarray]:
    """S = alpha * I + (1 - alpha) * T in float32 (see orc_combine_scores)."""
    imp = np.ascontiguousarray(importance, dtype=np.float32)
    tra = np.ascontiguousarray(transfer, dtype=np.float32)
    assert imp.shape == tra.shape
    out = np.zeros(imp.shape, dtype=np.float32)
    st = lib().orc_combine_scores(_ptr(imp), _ptr(tra), C.c_float(alpha), imp.size, _ptr(out))
    return st, out


def bits_from_features(features: np.ndarray, hidden: int, params: np.ndarray) -> Tuple[int, np.ndarray, np.ndarray]:
    """(status, bits [n], outputs [n, 4]) of the two-layer controller (see orc_bits_from_features).
    features: [n, 6]; params: W1 [hidden, 6], b1 [hidden], W2 [4, hidden], b2 [4] flattened in this order."""
    x = np.ascontiguousarray(features, dtype=np.float32).reshape(-1, 6)
    w = np.ascontiguousarray(params, dtype=np.float32).reshape(-1)
    assert w.size == 11 * hidden + 4
    bits = np.zeros(x.shape[0], dtype=np.uint8)
    outs = np.zeros((x.shape[0], 4), dtype=np.float32)
    st = lib().orc_bits_from_features(_ptr(x), x.shape[0], int(hidden), _ptr(w), _ptr(bits), _ptr(outs))
    return st, bits, outs


def num_threads() -> int:
    return int(lib().orc_num_threads())


def set_num_threads(n: int) -> None:
    lib().orc_set_num_threads(int(n))


HEADER_FIELDS = {  # name: (byte offset, numpy dtype) -- typed here from the oracle's own layout comment
    "magic": (0, "<u4"), "version": (4, "<u4"), "status": (8, "<u4"), "bits_mode": (12, "<u4"),
    "n_layers": (16, "<i4"), "n_kv_heads": (20, "<i4"), "head_dim": (24, "<i4"),
    "n_tokens": (28, "<i4"), "group_size": (32, "<i4"), "meta_bytes_per_group": (36, "<u4"),
    "model_id": (40, "<u8"), "sender_id": (48, "<u8"), "position_offset": (56, "<i8"),
    "sum_bits": (64, "<u8"), "avg_code_bits": (72, "<f4"), "bits_off": (80, "<u8"),
    "offs_off": (88, "<u8"), "payload_off": (96, "<u8"), "stream_bytes": (104, "<u8"),
    "total_bytes": (112, "<u8"), "sbase_off": (120, "<u8"),
}


def parse_header(card: np.ndarray) -> dict:
    raw = np.ascontiguousarray(card[:256], dtype=np.uint8)
    return {k: raw[o:o + np.dtype(dt).itemsize].view(dt)[0].item() for k, (o, dt) in HEADER_FIELDS.items()}
