"""QKVShare CacheCard create / inject for B200: thin Python face of the CUDA library.

`binding` marshals arguments into the C entry points of libqkvshare.so; `workloads` generates
the seeded synthetic caches and bit-width vectors; `build` compiles the library in-tree.
"""
from . import binding, workloads  # noqa: F401
from .binding import (CardHeader, CardMeta, Layout, QkvsError, attend_scratch_size, bits_from_features, bits_from_scores, bits_from_scores_budget, card_attend, combine_scores, card_create, card_info,  # noqa: F401
                      card_inject, card_inject_noalloc, card_prefix_size, card_send, card_size, layout_of, load_library,
                      make_layout, new_workspace, record_bytes, selftest_bounded_wait, selftest_division, status_string,
                      version)
