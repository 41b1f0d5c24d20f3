"""ctypes binding of libqkvshare.so: argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  PyTorch tensors are used as
device buffers and for the current stream; nothing here computes.  If the shared library is
missing the functions raise: there is no fallback implementation.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libqkvshare.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_BAD_BITS, ERR_BUFFER_TOO_SMALL, ERR_BAD_CARD, \
    ERR_CUDA, ERR_TIMEOUT = range(8)


class QkvsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class Layout(C.Structure):
    """qkvs_layout_t"""
    _fields_ = [("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_tokens", C.c_int32), ("group_size", C.c_int32), ("bits_mode", C.c_int32),
                ("head_stride", C.c_int64), ("token_stride", C.c_int64),
                ("meta_bytes", C.c_int32), ("reserved_", C.c_int32)]


class CardMeta(C.Structure):
    """qkvs_card_meta_t"""
    _fields_ = [("model_id", C.c_uint64), ("sender_id", C.c_uint64), ("position_offset", C.c_int64)]


class CardHeader(C.Structure):
    """qkvs_card_header_t"""
    _fields_ = [("magic", C.c_uint32), ("version", C.c_uint32), ("status", C.c_uint32),
                ("bits_mode", C.c_uint32), ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("n_tokens", C.c_int32), ("group_size", C.c_int32),
                ("meta_bytes_per_group", C.c_uint32), ("model_id", C.c_uint64),
                ("sender_id", C.c_uint64), ("position_offset", C.c_int64), ("sum_bits", C.c_uint64),
                ("avg_code_bits", C.c_float), ("pad0_", C.c_uint32), ("bits_off", C.c_uint64),
                ("offs_off", C.c_uint64), ("payload_off", C.c_uint64), ("stream_bytes", C.c_uint64),
                ("total_bytes", C.c_uint64), ("sbase_off", C.c_uint64), ("reserved_", C.c_uint8 * 128)]


assert C.sizeof(CardHeader) == 256

EXPORTS = ("qkvs_record_bytes", "qkvs_card_size", "qkvs_card_prefix_size", "qkvs_card_create",
           "qkvs_card_inject", "qkvs_card_inject_noalloc", "qkvs_card_send", "qkvs_attend_scratch_size", "qkvs_card_attend",
           "qkvs_card_info", "qkvs_bits_from_scores", "qkvs_bits_from_scores_budget", "qkvs_combine_scores", "qkvs_bits_from_features", "qkvs_selftest_division",
           "qkvs_selftest_bounded_wait", "qkvs_status_string",
           "qkvs_version")

_lib = None


def load_library(path: Optional[str] = None):
    """Load libqkvshare.so (built in-tree by paper_2605_03884_b200/build.py)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(
            f"{p} not found: build it with `python -m paper_2605_03884_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(p)
    vp = C.c_void_p
    lib.qkvs_record_bytes.restype = C.c_size_t
    lib.qkvs_record_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
    lib.qkvs_card_size.restype = C.c_int
    lib.qkvs_card_size.argtypes = [C.POINTER(Layout), vp, C.POINTER(C.c_size_t)]
    lib.qkvs_card_prefix_size.restype = C.c_int
    lib.qkvs_card_prefix_size.argtypes = [C.POINTER(Layout), C.POINTER(C.c_size_t)]
    lib.qkvs_card_create.restype = C.c_int
    lib.qkvs_card_create.argtypes = [C.POINTER(Layout), vp, vp, vp, C.POINTER(CardMeta), vp, C.c_size_t, vp, vp]
    lib.qkvs_card_inject.restype = C.c_int
    lib.qkvs_card_inject.argtypes = [vp, C.c_size_t, C.POINTER(Layout), vp, vp, C.c_int64, vp, vp]
    lib.qkvs_card_inject_noalloc.restype = C.c_int
    lib.qkvs_card_inject_noalloc.argtypes = [vp, C.c_size_t, C.POINTER(Layout), vp, vp, C.c_int64, vp, vp]
    lib.qkvs_card_send.restype = C.c_int
    lib.qkvs_card_send.argtypes = [vp, C.c_size_t, C.c_int32, vp, C.c_size_t, C.c_int32, vp]
    lib.qkvs_attend_scratch_size.restype = C.c_int
    lib.qkvs_attend_scratch_size.argtypes = [C.POINTER(Layout), C.c_int32, C.POINTER(C.c_size_t)]
    lib.qkvs_card_attend.restype = C.c_int
    lib.qkvs_card_attend.argtypes = [vp, C.c_size_t, C.POINTER(Layout), C.c_int32, vp, C.c_float, vp, vp, C.c_size_t, vp]
    lib.qkvs_bits_from_scores.restype = C.c_int
    lib.qkvs_bits_from_scores.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, vp]
    lib.qkvs_bits_from_scores_budget.restype = C.c_int
    lib.qkvs_bits_from_scores_budget.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_uint64, vp, vp, vp, vp, vp]
    lib.qkvs_combine_scores.restype = C.c_int
    lib.qkvs_combine_scores.argtypes = [vp, vp, C.c_float, C.c_int64, vp, vp]
    lib.qkvs_bits_from_features.restype = C.c_int
    lib.qkvs_bits_from_features.argtypes = [vp, C.c_int64, C.c_int32, vp, vp, vp, vp]
    lib.qkvs_card_info.restype = C.c_int
    lib.qkvs_card_info.argtypes = [vp, vp, C.POINTER(CardHeader)]
    lib.qkvs_selftest_division.restype = C.c_int
    lib.qkvs_selftest_division.argtypes = [vp, vp]
    lib.qkvs_selftest_bounded_wait.restype = C.c_int
    lib.qkvs_selftest_bounded_wait.argtypes = [C.c_uint32, vp, vp, vp]
    lib.qkvs_status_string.restype = C.c_char_p
    lib.qkvs_status_string.argtypes = [C.c_int]
    lib.qkvs_version.restype = C.c_int32
    if path is None:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().qkvs_status_string(int(status)).decode()


def make_layout(n_layers: int, n_kv_heads: int, head_dim: int, n_tokens: int, bits_mode: int = 0,
                head_stride: Optional[int] = None, token_stride: Optional[int] = None,
                meta_bytes: int = 8, group_size: int = 32) -> Layout:
    ts = head_dim if token_stride is None else token_stride
    hs = n_tokens * ts if head_stride is None else head_stride
    return Layout(n_layers, n_kv_heads, head_dim, n_tokens, group_size, bits_mode, hs, ts, meta_bytes, 0)


def layout_of(tensors: Sequence, n_tokens: Optional[int] = None, bits_mode: int = 0,
              meta_bytes: int = 8) -> Layout:
    """Layout of a list of per-layer torch tensors shaped [H, T_cap, d] or [1, H, T_cap, d]."""
    t = tensors[0]
    if t.dim() == 4:
        if t.shape[0] != 1:
            raise ValueError("batch size must be 1")
        t = t[0]
    if t.dim() != 3 or t.stride(2) != 1:
        raise ValueError("expected [H, T, d] with unit channel stride")
    h, tcap, d = t.shape
    return Layout(len(tensors), h, d, tcap if n_tokens is None else n_tokens, 32, bits_mode,
                  t.stride(0), t.stride(1), meta_bytes, 0)


def _ptr_array(tensors: Sequence):
    return (C.c_void_p * len(tensors))(*[int(t.data_ptr()) for t in tensors])


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def record_bytes(head_dim: int, b: int, meta_bytes: int = 8) -> int:
    return int(load_library().qkvs_record_bytes(head_dim, b, meta_bytes))


def card_size(layout: Layout, bits_host=None) -> int:
    """qkvs_card_size.  bits_host: numpy uint8 array / bytes on the host, or None (worst case)."""
    out = C.c_size_t(0)
    ptr = None
    keep = None
    if bits_host is not None:
        import numpy as np
        keep = np.ascontiguousarray(bits_host, dtype=np.uint8)
        ptr = keep.ctypes.data
    st = load_library().qkvs_card_size(C.byref(layout), ptr, C.byref(out))
    if st != OK:
        raise QkvsError(st, "qkvs_card_size")
    return int(out.value)


def card_prefix_size(layout: Layout) -> int:
    out = C.c_size_t(0)
    st = load_library().qkvs_card_prefix_size(C.byref(layout), C.byref(out))
    if st != OK:
        raise QkvsError(st, "qkvs_card_prefix_size")
    return int(out.value)


WORKSPACE_BYTES = 256


def new_workspace(device="cuda"):
    """A scratch block for card_create / card_inject: WORKSPACE_BYTES of device memory (int32)."""
    import torch
    return torch.zeros(WORKSPACE_BYTES // 4, dtype=torch.int32, device=device)


def _workspace_ptr(workspace):
    if workspace is None:
        return None
    if workspace.numel() * workspace.element_size() < WORKSPACE_BYTES:
        raise ValueError(f"workspace must hold {WORKSPACE_BYTES} bytes")
    return int(workspace.data_ptr())


def card_create(layout: Layout, K_layers: Sequence, V_layers: Sequence, bits_dev, card_dev,
                meta: Optional[CardMeta] = None, card_capacity: Optional[int] = None,
                workspace=None, stream=None, check: bool = True, src_token_offset: int = 0) -> int:
    """qkvs_card_create.  K_layers / V_layers: per-layer CUDA tensors (FP16); bits_dev: CUDA uint8
    tensor; card_dev: CUDA uint8 tensor that receives the card; workspace: CUDA tensor of
    WORKSPACE_BYTES bytes (see new_workspace) or None.  src_token_offset: the cache row that
    becomes token 0 of the card (the library is handed pointers to that row; layout.n_tokens rows
    from there are encoded) -- a card of only the tokens appended since the last one.  Returns
    the status."""
    lib = load_library()
    kp, vp = _ptr_array(K_layers), _ptr_array(V_layers)
    if src_token_offset:
        step = int(src_token_offset) * int(layout.token_stride) * 2  # FP16 elements
        kp = (C.c_void_p * len(K_layers))(*[int(t.data_ptr()) + step for t in K_layers])
        vp = (C.c_void_p * len(V_layers))(*[int(t.data_ptr()) + step for t in V_layers])
    cap = int(card_dev.numel() * card_dev.element_size()) if card_capacity is None else int(card_capacity)
    st = lib.qkvs_card_create(C.byref(layout), kp, vp, int(bits_dev.data_ptr()) if bits_dev is not None else None,
                              C.byref(meta) if meta is not None else None, int(card_dev.data_ptr()), cap,
                              _workspace_ptr(workspace), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_card_create")
    return st


def card_inject(card_dev, dst_layout: Layout, K_out: Sequence, V_out: Sequence,
                dst_token_offset: int = 0, card_bytes: Optional[int] = None, workspace=None,
                stream=None, check: bool = True) -> int:
    """qkvs_card_inject.  workspace: CUDA int32 tensor of WORKSPACE_BYTES bytes or None; after
    the call its element 0 is the status word the kernel recorded."""
    lib = load_library()
    kp, vp = _ptr_array(K_out), _ptr_array(V_out)
    nbytes = int(card_dev.numel() * card_dev.element_size()) if card_bytes is None else int(card_bytes)
    st = lib.qkvs_card_inject(int(card_dev.data_ptr()), nbytes, C.byref(dst_layout), kp, vp,
                              int(dst_token_offset),
                              _workspace_ptr(workspace), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_card_inject")
    return st


NOALLOC_MAX_LAYERS = 4096


def card_inject_noalloc(card_dev, dst_layout: Layout, K_out: Sequence, V_out: Sequence,
                        dst_token_offset: int = 0, card_bytes: Optional[int] = None, status_dev=None,
                        stream=None, check: bool = True) -> int:
    """qkvs_card_inject_noalloc: injection whose work counters sit in the library's own device
    memory, for callers that may not allocate a scratch block.  status_dev: optional CUDA int32
    tensor of one element.  Calls on one GPU must not overlap in time."""
    lib = load_library()
    kp, vp = _ptr_array(K_out), _ptr_array(V_out)
    nbytes = int(card_dev.numel() * card_dev.element_size()) if card_bytes is None else int(card_bytes)
    st = lib.qkvs_card_inject_noalloc(int(card_dev.data_ptr()), nbytes, C.byref(dst_layout), kp, vp,
                                      int(dst_token_offset),
                                      int(status_dev.data_ptr()) if status_dev is not None else None,
                                      _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_card_inject_noalloc")
    return st


def card_send(card_dev, dst_dev, card_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """qkvs_card_send: copies a card (CUDA uint8 tensor) into `dst_dev`, a CUDA uint8 tensor on the
    same or on another GPU; the devices are taken from the tensors."""
    nbytes = int(card_dev.numel() * card_dev.element_size()) if card_bytes is None else int(card_bytes)
    st = load_library().qkvs_card_send(int(card_dev.data_ptr()), nbytes, int(card_dev.device.index),
                                       int(dst_dev.data_ptr()), int(dst_dev.numel() * dst_dev.element_size()),
                                       int(dst_dev.device.index), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_card_send")
    return st


def attend_scratch_size(layout: Layout, n_q_heads: int) -> int:
    out = C.c_size_t(0)
    st = load_library().qkvs_attend_scratch_size(C.byref(layout), int(n_q_heads), C.byref(out))
    if st != OK:
        raise QkvsError(st, "qkvs_attend_scratch_size")
    return int(out.value)


def card_attend(card_dev, layout: Layout, q_dev, out_dev, scratch_dev, softmax_scale: Optional[float] = None,
                card_bytes: Optional[int] = None, stream=None, check: bool = True) -> int:
    """qkvs_card_attend.  q_dev: CUDA FP16 [L, n_q_heads, d]; out_dev: CUDA FP32 of the same
    shape; scratch_dev: CUDA uint8 tensor of attend_scratch_size() bytes (its first int32 is the
    status word afterwards).  softmax_scale defaults to 1/sqrt(d)."""
    nbytes = int(card_dev.numel() * card_dev.element_size()) if card_bytes is None else int(card_bytes)
    scale = float(layout.head_dim) ** -0.5 if softmax_scale is None else float(softmax_scale)
    st = load_library().qkvs_card_attend(int(card_dev.data_ptr()), nbytes, C.byref(layout), int(q_dev.shape[1]),
                                         int(q_dev.data_ptr()), scale, int(out_dev.data_ptr()),
                                         int(scratch_dev.data_ptr()),
                                         int(scratch_dev.numel() * scratch_dev.element_size()), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_card_attend")
    return st


def bits_from_scores(scores_dev, n_fp16: int, n_8bit: int, n_4bit: int, bits_dev, stream=None, check: bool = True) -> int:
    """qkvs_bits_from_scores.  scores_dev: CUDA float32 [T] or [n_segments, T]; bits_dev: CUDA uint8
    of the same shape."""
    n_seg = 1 if scores_dev.dim() == 1 else int(scores_dev.shape[0])
    n_tok = int(scores_dev.shape[-1])
    st = load_library().qkvs_bits_from_scores(int(scores_dev.data_ptr()), n_seg, n_tok, int(n_fp16), int(n_8bit),
                                              int(n_4bit), int(bits_dev.data_ptr()), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_bits_from_scores")
    return st


def bits_from_scores_budget(scores_dev, head_dim: int, budget_bytes: int, bits_dev, weights=None, meta_bytes: int = 8,
                            offsets_dev=None, status_dev=None, stream=None, check: bool = True) -> int:
    """qkvs_bits_from_scores_budget.  scores_dev: CUDA float32 [T] or [n_segments, T]; bits_dev: CUDA
    uint8 of the same shape; weights: three floats or None; offsets_dev: optional CUDA int32/uint32
    [n_segments, T + 1]; status_dev: optional CUDA int32 of one element."""
    n_seg = 1 if scores_dev.dim() == 1 else int(scores_dev.shape[0])
    n_tok = int(scores_dev.shape[-1])
    w = (C.c_float * 3)(*[float(x) for x in weights]) if weights is not None else None
    st = load_library().qkvs_bits_from_scores_budget(
        int(scores_dev.data_ptr()), n_seg, n_tok, int(head_dim), int(meta_bytes), int(budget_bytes), w,
        int(bits_dev.data_ptr()), int(offsets_dev.data_ptr()) if offsets_dev is not None else None,
        int(status_dev.data_ptr()) if status_dev is not None else None, _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_bits_from_scores_budget")
    return st


def combine_scores(importance_dev, transfer_dev, alpha: float, scores_dev, stream=None, check: bool = True) -> int:
    """qkvs_combine_scores: scores = alpha * importance + (1 - alpha) * transfer, CUDA float32 tensors
    of equal size."""
    n = int(importance_dev.numel())
    st = load_library().qkvs_combine_scores(int(importance_dev.data_ptr()), int(transfer_dev.data_ptr()), C.c_float(alpha),
                                            n, int(scores_dev.data_ptr()), _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_combine_scores")
    return st


def bits_from_features(features_dev, hidden: int, params_dev, bits_dev, outputs_dev=None, stream=None, check: bool = True) -> int:
    """qkvs_bits_from_features.  features_dev: CUDA float32 [n, 6]; params_dev: CUDA float32 of
    11 * hidden + 4 elements (W1, b1, W2, b2); bits_dev: CUDA uint8 [n]; outputs_dev: optional CUDA
    float32 [n, 4]."""
    n = int(features_dev.shape[0])
    st = load_library().qkvs_bits_from_features(
        int(features_dev.data_ptr()), n, int(hidden), int(params_dev.data_ptr()), int(bits_dev.data_ptr()),
        int(outputs_dev.data_ptr()) if outputs_dev is not None else None, _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_bits_from_features")
    return st


def card_info(card_dev, stream=None):
    """qkvs_card_info -> (status, CardHeader).  Synchronises the stream."""
    hdr = CardHeader()
    st = load_library().qkvs_card_info(int(card_dev.data_ptr()), _stream_handle(stream), C.byref(hdr))
    return st, hdr


def selftest_division(mismatches_dev, stream=None) -> int:
    """qkvs_selftest_division.  mismatches_dev: CUDA int64 tensor of two elements."""
    st = load_library().qkvs_selftest_division(int(mismatches_dev.data_ptr()), _stream_handle(stream))
    if st != OK:
        raise QkvsError(st, "qkvs_selftest_division")
    return st


def selftest_bounded_wait(limit_us: int, status_dev, waited_ns_dev=None, stream=None, check: bool = True) -> int:
    """qkvs_selftest_bounded_wait.  status_dev: CUDA int32 tensor of one element; waited_ns_dev:
    optional CUDA int64 tensor of one element."""
    st = load_library().qkvs_selftest_bounded_wait(int(limit_us), int(status_dev.data_ptr()),
                                                   int(waited_ns_dev.data_ptr()) if waited_ns_dev is not None else None,
                                                   _stream_handle(stream))
    if check and st != OK:
        raise QkvsError(st, "qkvs_selftest_bounded_wait")
    return st


def version() -> int:
    return int(load_library().qkvs_version())
