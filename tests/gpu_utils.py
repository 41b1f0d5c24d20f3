"""Helpers for the GPU parity tests: run the CUDA path on numpy inputs, compare with the oracle."""
from __future__ import annotations

import numpy as np

POISON = 0xA5
PAD = 512


def ulp_key(h16: np.ndarray) -> np.ndarray:
    """FP16 bit patterns -> integers whose difference counts representable values between two
    numbers (sign-magnitude folded onto a line; +0 and -0 coincide)."""
    u = h16.view(np.uint16).astype(np.int32)
    mag = u & 0x7fff
    return np.where(u & 0x8000, -mag, mag)


def max_ulp(a: np.ndarray, b: np.ndarray) -> int:
    if a.size == 0:
        return 0
    return int(np.abs(ulp_key(a) - ulp_key(b)).max())


def padded_cache(L, H, T, d, seed, t_cap=None, token_stride=None, scale=2.0):
    """Per-layer K, V numpy arrays [H, t_cap, token_stride] whose [:, :T, :d] part holds data."""
    t_cap = T if t_cap is None else t_cap
    ts = d if token_stride is None else token_stride
    rng = np.random.default_rng(seed)
    Ks, Vs = [], []
    for _ in range(L):
        for dst in (Ks, Vs):
            buf = np.full((H, t_cap, ts), 777.0, dtype=np.float16)
            buf[:, :T, :d] = (rng.standard_normal((H, T, d), dtype=np.float32) * scale).astype(np.float16)
            dst.append(buf)
    return Ks, Vs, dict(head_stride=t_cap * ts, token_stride=ts)


def to_cuda(arrs):
    import torch
    return [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in arrs]


def dirty_workspace(q):
    """A scratch block filled with junk: the calls must not depend on what it holds on entry."""
    import torch
    ws = q.new_workspace()
    ws.fill_(0x5A5A5A5A)
    return ws


def gpu_create(q, lay, Ks, Vs, bits, meta=None, capacity=None, Kd=None, Vd=None, scratch=True):
    """Run qkvs_card_create into a poisoned buffer; returns (status_from_header, card_bytes_np,
    whole_buffer_np, capacity).  The buffer has PAD canary bytes behind `capacity`.  `scratch`
    False passes no scratch block (work is then split in advance)."""
    import torch
    Kd = to_cuda(Ks) if Kd is None else Kd
    Vd = to_cuda(Vs) if Vd is None else Vd
    bits_d = torch.from_numpy(np.ascontiguousarray(bits, dtype=np.uint8)).cuda()
    cap = q.card_size(lay, None) if capacity is None else capacity
    buf = torch.full((cap + PAD,), POISON, dtype=torch.uint8, device="cuda")
    q.card_create(lay, Kd, Vd, bits_d, buf, meta=meta, card_capacity=cap,
                  workspace=dirty_workspace(q) if scratch else None)
    st, hdr = q.card_info(buf)
    torch.cuda.synchronize()
    whole = buf.cpu().numpy()
    return st, hdr, whole, cap


def gpu_inject(q, card_np, dst_lay, Ko_np, Vo_np, dst_token_offset=0, card_bytes=None, scratch=True):
    """Upload a card and destination buffers, inject, return (device status, K_out, V_out).
    Without a scratch block there is no status word; None is returned in its place."""
    import torch
    card_d = torch.from_numpy(np.ascontiguousarray(card_np)).cuda()
    Kd, Vd = to_cuda(Ko_np), to_cuda(Vo_np)
    ws = dirty_workspace(q) if scratch else None
    q.card_inject(card_d, dst_lay, Kd, Vd, dst_token_offset=dst_token_offset,
                  card_bytes=card_np.size if card_bytes is None else card_bytes, workspace=ws)
    torch.cuda.synchronize()
    status = int(ws[0].item()) if scratch else None
    return status, [k.cpu().numpy() for k in Kd], [v.cpu().numpy() for v in Vd]
