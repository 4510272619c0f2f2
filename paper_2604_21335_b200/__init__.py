"""B200-native decode attention over a Quest-selected, value-group-routed KV cache.

The product is ``libstc.so`` (hand-written CUDA for sm_100a behind a C ABI,
declared in ``include/stc.h``).  :mod:`paper_2604_21335_b200.binding` marshals
torch tensors into those calls; it does no arithmetic of its own and raises if
the library is missing -- there is no fallback path.
"""
from . import binding, workload  # noqa: F401
from .binding import (  # noqa: F401
    StcError, Shape, Cache, build_page_meta, quest_select, route_pack, decode_attn,
    workspace_bytes, cache_bytes, load_library, pass_host, pass_host_arena_bytes, quest_select_static, route_mask, pack_values, append_tokens, router_logits, query_bias, pages_to_class, route_new_pages, decode_step, decode_step_host, decode_step_host_arena_bytes,
)
