"""qkvs_card_inject_noalloc against qkvs_card_inject, through the C-ABI, on a B200.

Some receivers cannot hand the library a scratch block: a component of a serving engine that has
given all free GPU memory to its KV-cache pool may not call cudaMalloc at all.  For them the
library keeps the work counters in a small array of its own.  That array is shared by every call
and still holds the previous call's counts when the next one starts, so the test injects several
times in a row -- cards of different shapes -- and wants every result to equal what the ordinary
entry point writes.

This file is collected last on purpose (a run that stops at the first failure has then already
run everything else), and it has to pass on its own in a fresh process as well as after the
other tests.
"""
import numpy as np
import pytest

import paper_2605_03884_b200 as q
from paper_2605_03884_b200 import build as qbuild
from paper_2605_03884_b200 import workloads as wl
from gpu_utils import max_ulp, padded_cache, to_cuda

pytestmark = pytest.mark.gpu

MAX_ULP = 1  # the tolerance of the parity tests for injected FP16 values


@pytest.fixture(scope="module", autouse=True)
def _library():
    qbuild.build()
    q.load_library()


def _make_card(L, H, d, T, seed):
    import torch
    Ks, Vs, _ = padded_cache(L, H, T, d, seed=seed)
    bits = wl.iid_bits(T, (0.4, 0.4, 0.15, 0.05), seed=seed + 1)
    lay = q.make_layout(L, H, d, T)
    card = torch.zeros(q.card_size(lay, bits), dtype=torch.uint8, device="cuda")
    q.card_create(lay, to_cuda(Ks), to_cuda(Vs), torch.from_numpy(bits).cuda(), card, workspace=q.new_workspace())
    st, _ = q.card_info(card)
    assert st == 0
    return lay, card


def _inject_both_ways(lay, card, L, H, d, T):
    import torch
    want_k = [torch.full((H, T, d), -3.0, dtype=torch.float16, device="cuda") for _ in range(L)]
    want_v = [torch.full((H, T, d), -5.0, dtype=torch.float16, device="cuda") for _ in range(L)]
    got_k = [t.clone() for t in want_k]
    got_v = [t.clone() for t in want_v]
    ws = q.new_workspace()
    q.card_inject(card, lay, want_k, want_v, workspace=ws)
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    st = q.card_inject_noalloc(card, lay, got_k, got_v, status_dev=status)
    torch.cuda.synchronize()
    assert st == 0 and int(ws[0].item()) == 0 and int(status.item()) == 0
    worst = 0
    for g, w in zip(got_k + got_v, want_k + want_v):
        worst = max(worst, max_ulp(g.cpu().numpy(), w.cpu().numpy()))
    return worst


def test_calls_in_a_row_match_the_ordinary_entry_point():
    # first call: enough chunks that every warp goes back to the counter several times
    L, H, d, T = 4, 8, 128, 9000
    lay, card = _make_card(L, H, d, T, seed=501)
    assert _inject_both_ways(lay, card, L, H, d, T) <= MAX_ULP
    # second call, straight after, another shape: the array still holds the first call's counts
    L2, H2, d2, T2 = 2, 3, 64, 777
    lay2, card2 = _make_card(L2, H2, d2, T2, seed=502)
    assert _inject_both_ways(lay2, card2, L2, H2, d2, T2) <= MAX_ULP
    # and the first one again
    assert _inject_both_ways(lay, card, L, H, d, T) <= MAX_ULP


def test_a_call_of_several_launches_uses_the_higher_counters():
    """More than 64 layers make more than one kernel launch per call, each with a counter of its
    own further up the array; run after a large call, so that those words start out non-zero
    only if a launch left them so, and twice, so that the second run meets the first one's counts."""
    L, H, d, T = 130, 1, 64, 300
    lay, card = _make_card(L, H, d, T, seed=503)
    assert _inject_both_ways(lay, card, L, H, d, T) <= MAX_ULP
    assert _inject_both_ways(lay, card, L, H, d, T) <= MAX_ULP


def test_more_layers_than_the_array_has_counters_for_is_refused():
    import torch
    L = q.binding.NOALLOC_MAX_LAYERS + 1
    lay = q.make_layout(L, 1, 64, 16)
    card = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    one = torch.zeros((1, 16, 64), dtype=torch.float16, device="cuda")
    st = q.card_inject_noalloc(card, lay, [one] * L, [one] * L, check=False)
    assert st == q.binding.ERR_UNSUPPORTED_SHAPE
    assert torch.count_nonzero(one).item() == 0
