"""ctypes binding of libstc.so: argument marshalling only.

Every function takes CUDA tensors, checks dtype / contiguity / device, and
passes ``data_ptr()`` plus the current stream to the C-ABI call of the same
name.  No step of the method runs in Python, and there is no CPU fallback: if
the shared library is missing the import of the library fails loudly.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from pathlib import Path
from typing import Optional

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libstc.so"

OP_QUEST_SELECT, OP_ROUTE_PACK, OP_DECODE_ATTN = 1, 2, 3
MODE_GLOBAL, MODE_PER_TOKEN = 0, 1
CLS_DROP, CLS_ROUTED, CLS_FULL = 0, 1, 2
STC_OK = 0
STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = (
    "stc_status_string", "stc_version", "stc_workspace_bytes", "stc_build_page_meta",
    "stc_quest_select", "stc_route_pack", "stc_decode_attn", "stc_cache_bytes",
    "stc_pass_host_arena_bytes", "stc_pass_host", "stc_quest_select_static", "stc_route_mask", "stc_pack_values", "stc_append_tokens", "stc_router_logits", "stc_query_bias", "stc_quest_select_window", "stc_pages_to_class", "stc_route_new_pages", "stc_decode_step", "stc_decode_step_host_arena_bytes", "stc_decode_step_host",
)


class StcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().stc_status_string(code).decode()
        super().__init__(f"{where}: {msg} (status {code})")


class _Shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("page_size", C.c_int32), ("n_groups", C.c_int32),
                ("t_cap", C.c_int32), ("reserved", C.c_int32), ("seq_len", C.c_void_p)]


class _Cache(C.Structure):
    _fields_ = [("k", C.c_void_p), ("kmin", C.c_void_p), ("kmax", C.c_void_p),
                ("v_packed", C.c_void_p), ("v_mask", C.c_void_p), ("v_offs", C.c_void_p),
                ("cap_groups", C.c_int64)]


_lib = None


def load_library():
    """Load libstc.so (built in-tree by ``paper_2604_21335_b200.build``)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2604_21335_b200.build` "
                "(nvcc, sm_100a).  There is no fallback implementation.")
        lib = C.CDLL(str(_LIB_PATH))
        lib.stc_status_string.restype = C.c_char_p
        lib.stc_status_string.argtypes = [C.c_int32]
        lib.stc_version.restype = C.c_int32
        for name in EXPORTS[2:]:
            getattr(lib, name).restype = C.c_int32
        lib.stc_workspace_bytes.argtypes = [C.POINTER(_Shape), C.c_int32, C.c_int64, C.POINTER(C.c_size_t)]
        lib.stc_build_page_meta.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_int32, C.c_int32, C.c_void_p]
        lib.stc_quest_select.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_int32, C.c_int32,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        lib.stc_quest_select_window.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_int32, C.c_int32,
                                                C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                                C.c_void_p]
        lib.stc_quest_select_static.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_int32,
                                                C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_pages_to_class.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                           C.c_void_p]
        lib.stc_route_pack.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                       C.c_int32, C.c_int32, C.c_int32, C.POINTER(_Cache), C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        lib.stc_route_mask.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                       C.c_int32, C.POINTER(_Cache), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.stc_pack_values.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_int32, C.POINTER(_Cache), C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        lib.stc_append_tokens.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_route_new_pages.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_void_p, C.c_int32,
                                            C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_query_bias.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_router_logits.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_decode_attn.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
        lib.stc_decode_step.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
        lib.stc_cache_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        lib.stc_pass_host_arena_bytes.argtypes = [C.POINTER(_Shape), C.c_int64, C.c_int32, C.POINTER(C.c_size_t)]
        lib.stc_pass_host.argtypes = [C.POINTER(_Shape), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_int64,
                                      C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.stc_decode_step_host_arena_bytes.argtypes = [C.POINTER(_Shape), C.c_int32, C.POINTER(C.c_size_t)]
        lib.stc_decode_step_host.argtypes = [C.POINTER(_Shape), C.POINTER(_Cache), C.c_void_p, C.c_int32, C.c_float,
                                             C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Shape:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    n_groups: int
    t_cap: int
    seq_len: Optional[torch.Tensor] = None   # int32 [batch] on the device, or None
    head_dim: int = 128
    page_size: int = 16

    @property
    def n_pages(self) -> int:
        return (self.t_cap + self.page_size - 1) // self.page_size

    @property
    def n_problems(self) -> int:
        return self.batch * self.n_kv_heads

    def c(self) -> _Shape:
        sl = _ptr(self.seq_len, torch.int32, "seq_len")
        return _Shape(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.page_size,
                      self.n_groups, self.t_cap, 0, sl)


@dataclass
class Cache:
    k: Optional[torch.Tensor] = None          # bf16 [B,Hkv,T,128]
    kmin: Optional[torch.Tensor] = None       # bf16 [B,Hkv,P,128]
    kmax: Optional[torch.Tensor] = None
    v_packed: Optional[torch.Tensor] = None   # bf16 [B,Hkv,cap_groups,128/S]
    v_mask: Optional[torch.Tensor] = None     # int16/uint16 [B,Hkv,T]
    v_offs: Optional[torch.Tensor] = None     # int32/uint32 [B,Hkv,T+1]
    cap_groups: int = 0

    def c(self) -> _Cache:
        return _Cache(_ptr(self.k, torch.bfloat16, "k"), _ptr(self.kmin, torch.bfloat16, "kmin"),
                      _ptr(self.kmax, torch.bfloat16, "kmax"), _ptr(self.v_packed, torch.bfloat16, "v_packed"),
                      _ptr(self.v_mask, None, "v_mask"), _ptr(self.v_offs, None, "v_offs"), self.cap_groups)

    @staticmethod
    def allocate(shape: Shape, k: torch.Tensor, cap_groups: int) -> "Cache":
        """Device buffers for the metadata and the packed store (torch owns the memory)."""
        dev = k.device
        B, H, T, P = shape.batch, shape.n_kv_heads, shape.t_cap, shape.n_pages
        g = shape.head_dim // shape.n_groups
        return Cache(
            k=k,
            kmin=torch.empty(B, H, P, shape.head_dim, dtype=torch.bfloat16, device=dev),
            kmax=torch.empty(B, H, P, shape.head_dim, dtype=torch.bfloat16, device=dev),
            v_packed=torch.empty(B, H, max(cap_groups, 1), g, dtype=torch.bfloat16, device=dev),
            v_mask=torch.zeros(B, H, T, dtype=torch.int16, device=dev),
            v_offs=torch.zeros(B, H, T + 1, dtype=torch.int32, device=dev),
            cap_groups=cap_groups)


def _check(rc: int, where: str):
    if rc != STC_OK:
        raise StcError(rc, where)


def workspace_bytes(shape: Shape, op: int, arg: int = 0) -> int:
    out = C.c_size_t(0)
    cs = shape.c()
    _check(load_library().stc_workspace_bytes(C.byref(cs), op, arg, C.byref(out)), "stc_workspace_bytes")
    return int(out.value)


def new_workspace(shape: Shape, op: int, arg: int = 0, device="cuda") -> torch.Tensor:
    n = workspace_bytes(shape, op, arg)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device)


def build_page_meta(shape: Shape, cache: Cache, page_begin: int = 0, page_end: int = -1) -> None:
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_build_page_meta(C.byref(cs), C.byref(cc), page_begin, page_end, _stream()),
           "stc_build_page_meta")


def quest_select(shape: Shape, cache: Cache, q: torch.Tensor, token_budget: int, page_ids: torch.Tensor,
                 n_pages: torch.Tensor, ws: torch.Tensor, scores: Optional[torch.Tensor] = None,
                 n_recent_pages: int = 0) -> None:
    """n_recent_pages > 0 keeps that many most recent pages unconditionally (stc_quest_select_window)."""
    cs, cc = shape.c(), cache.c()
    if n_recent_pages:
        _check(load_library().stc_quest_select_window(
            C.byref(cs), C.byref(cc), _ptr(q, torch.bfloat16, "q"), token_budget, n_recent_pages,
            page_ids.shape[-1], _ptr(page_ids, torch.int32, "page_ids"), _ptr(n_pages, torch.int32, "n_pages"),
            _ptr(scores, torch.float32, "scores"), _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()),
            "stc_quest_select_window")
        return
    _check(load_library().stc_quest_select(
        C.byref(cs), C.byref(cc), _ptr(q, torch.bfloat16, "q"), token_budget, page_ids.shape[-1],
        _ptr(page_ids, torch.int32, "page_ids"), _ptr(n_pages, torch.int32, "n_pages"),
        _ptr(scores, torch.float32, "scores"), _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()),
        "stc_quest_select")


def quest_select_static(shape: Shape, cache: Cache, q: torch.Tensor, token_budget: int, page_ids: torch.Tensor,
                        n_pages: torch.Tensor, scores: Optional[torch.Tensor] = None) -> None:
    """stc_quest_select without a workspace argument: for callers that cannot
    allocate device memory where they select pages.  The scratch space is an array
    inside the library (STATIC_SCRATCH_BYTES per GPU); larger shapes raise StcError
    with code 8.  Calls must not overlap on the device."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_quest_select_static(
        C.byref(cs), C.byref(cc), _ptr(q, torch.bfloat16, "q"), token_budget, page_ids.shape[-1],
        _ptr(page_ids, torch.int32, "page_ids"), _ptr(n_pages, torch.int32, "n_pages"),
        _ptr(scores, torch.float32, "scores"), _stream()), "stc_quest_select_static")


def pages_to_class(shape: Shape, page_ids: torch.Tensor, n_pages: torch.Tensor, tok_class: torch.Tensor) -> None:
    """tok_class u8 [B,Hkv,T] <- ROUTED for the valid tokens of the listed pages, DROP elsewhere."""
    cs = shape.c()
    _check(load_library().stc_pages_to_class(
        C.byref(cs), _ptr(page_ids, torch.int32, "page_ids"), _ptr(n_pages, torch.int32, "n_pages"),
        page_ids.shape[-1], _ptr(tok_class, torch.uint8, "tok_class"), _stream()), "stc_pages_to_class")


def route_pack(shape: Shape, v: torch.Tensor, scores: torch.Tensor, tok_class: Optional[torch.Tensor],
               k_nominal: int, cache: Cache, total_groups: torch.Tensor, status: torch.Tensor,
               ws: torch.Tensor, min_per_token: int = 1, mode: int = MODE_GLOBAL) -> None:
    stride = 0
    if tok_class is not None and tok_class.dim() == 3:
        stride = shape.t_cap
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_route_pack(
        C.byref(cs), _ptr(v, torch.bfloat16, "v"), _ptr(scores, torch.float32, "scores"),
        _ptr(tok_class, torch.uint8, "tok_class"), stride, k_nominal, min_per_token, mode, C.byref(cc),
        _ptr(total_groups, torch.int64, "total_groups"), _ptr(status, torch.int32, "status"),
        _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()), "stc_route_pack")


def route_mask(shape: Shape, scores: torch.Tensor, tok_class: Optional[torch.Tensor], k_nominal: int,
               cache: Cache, ws: torch.Tensor, min_per_token: int = 1, mode: int = MODE_GLOBAL) -> None:
    """First half of route_pack: the routing masks (ties at the threshold are left in `ws`)."""
    stride = shape.t_cap if (tok_class is not None and tok_class.dim() == 3) else 0
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_route_mask(
        C.byref(cs), _ptr(scores, torch.float32, "scores"), _ptr(tok_class, torch.uint8, "tok_class"), stride,
        k_nominal, min_per_token, mode, C.byref(cc), _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()),
        "stc_route_mask")


def pack_values(shape: Shape, v: torch.Tensor, cache: Cache, total_groups: torch.Tensor, status: torch.Tensor,
                ws: torch.Tensor, mode: int = MODE_GLOBAL) -> None:
    """Second half of route_pack: final masks, offsets and the packed value store."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_pack_values(
        C.byref(cs), _ptr(v, torch.bfloat16, "v"), mode, C.byref(cc),
        _ptr(total_groups, torch.int64, "total_groups"), _ptr(status, torch.int32, "status"),
        _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()), "stc_pack_values")


def append_tokens(shape: Shape, cache: Cache, v: torch.Tensor, old_len: torch.Tensor, max_new: int,
                  total_groups: torch.Tensor, status: torch.Tensor) -> None:
    """Tokens old_len[b] .. shape.seq_len[b] were just added: store their values in full, refresh page metadata."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_append_tokens(
        C.byref(cs), C.byref(cc), _ptr(v, torch.bfloat16, "v"), _ptr(old_len, torch.int32, "old_len"), max_new,
        _ptr(total_groups, torch.int64, "total_groups"), _ptr(status, torch.int32, "status"), _stream()),
        "stc_append_tokens")


def route_new_pages(shape: Shape, cache: Cache, scores: torch.Tensor, first_page: torch.Tensor, k_nominal: int,
                    total_groups: torch.Tensor, status: torch.Tensor, min_per_token: int = 1,
                    mode: int = MODE_GLOBAL) -> None:
    """Routes, page by page, the complete pages from first_page[b] on (stored at full width by append_tokens)."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_route_new_pages(
        C.byref(cs), C.byref(cc), _ptr(scores, torch.float32, "scores"), _ptr(first_page, torch.int32, "first_page"),
        k_nominal, min_per_token, mode, _ptr(total_groups, torch.int64, "total_groups"),
        _ptr(status, torch.int32, "status"), _stream()), "stc_route_new_pages")


def router_logits(shape: Shape, h: torch.Tensor, w: torch.Tensor, scores: torch.Tensor, status_word: torch.Tensor,
                  bias: Optional[torch.Tensor] = None) -> None:
    """scores[b,hk,t,j] = h[b,t,:] . w[hk*S+j,:] (+ bias[b,hk*S+j]); h bf16 [B,T,d_model], w bf16 [Hkv*S,d_model]."""
    cs = shape.c()
    _check(load_library().stc_router_logits(
        C.byref(cs), _ptr(h, torch.bfloat16, "h"), _ptr(w, torch.bfloat16, "w"), _ptr(bias, torch.float32, "bias"),
        h.shape[-1], _ptr(scores, torch.float32, "scores"), _ptr(status_word, torch.int32, "status_word"),
        _stream()), "stc_router_logits")


def query_bias(h_q: torch.Tensor, w_q: torch.Tensor, s_q: torch.Tensor, bias: torch.Tensor,
               q_len: Optional[torch.Tensor] = None) -> None:
    """s_q[b,:] = mean of h_q[b,:q_len[b],:]; bias[b,n] = s_q[b,:] . w_q[n,:]; h_q bf16 [B,Lq,d_model], w_q bf16 [N,d_model]."""
    B, Lq, dm = h_q.shape
    _check(load_library().stc_query_bias(
        B, Lq, dm, w_q.shape[0], _ptr(h_q, torch.bfloat16, "h_q"), _ptr(q_len, torch.int32, "q_len"),
        _ptr(w_q, torch.bfloat16, "w_q"), _ptr(s_q, torch.float32, "s_q"), _ptr(bias, torch.float32, "bias"),
        _stream()), "stc_query_bias")


def decode_attn(shape: Shape, cache: Cache, q: torch.Tensor, page_ids: Optional[torch.Tensor],
                n_pages: Optional[torch.Tensor], sm_scale: float, out: torch.Tensor, ws: torch.Tensor,
                lse: Optional[torch.Tensor] = None) -> None:
    max_pages = page_ids.shape[-1] if page_ids is not None else shape.n_pages
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_decode_attn(
        C.byref(cs), C.byref(cc), _ptr(q, torch.bfloat16, "q"), _ptr(page_ids, torch.int32, "page_ids"),
        _ptr(n_pages, torch.int32, "n_pages"), max_pages, sm_scale, _ptr(out, torch.float32, "out"),
        _ptr(lse, torch.float32, "lse"), _ptr(ws, torch.uint8, "ws"), ws.numel(), _stream()),
        "stc_decode_attn")


def decode_step(shape: Shape, cache: Cache, q: torch.Tensor, token_budget: int, page_ids: torch.Tensor,
                n_pages: torch.Tensor, sm_scale: float, out: torch.Tensor, ws_select: torch.Tensor,
                ws_attn: torch.Tensor, lse: Optional[torch.Tensor] = None) -> None:
    """quest_select + decode_attn as one call (both workspaces cleared up front, the kernels back to back)."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_decode_step(
        C.byref(cs), C.byref(cc), _ptr(q, torch.bfloat16, "q"), token_budget, page_ids.shape[-1],
        _ptr(page_ids, torch.int32, "page_ids"), _ptr(n_pages, torch.int32, "n_pages"), sm_scale,
        _ptr(out, torch.float32, "out"), _ptr(lse, torch.float32, "lse"), _ptr(ws_select, torch.uint8, "ws_select"),
        ws_select.numel(), _ptr(ws_attn, torch.uint8, "ws_attn"), ws_attn.numel(), _stream()), "stc_decode_step")


def cache_bytes(n_tokens_retained: int, n_groups_kept: int, n_groups: int):
    """(key + packed value bytes, mask + offset + page-metadata bytes) of the compressed cache."""
    kv, idx = C.c_int64(0), C.c_int64(0)
    _check(load_library().stc_cache_bytes(n_tokens_retained, n_groups_kept, n_groups, C.byref(kv), C.byref(idx)),
           "stc_cache_bytes")
    return int(kv.value), int(idx.value)


def _hptr(t: Optional[torch.Tensor], dtype, name):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
        raise ValueError(f"{name} must be a contiguous host tensor of {dtype}")
    return C.c_void_p(t.data_ptr())


def pass_host_arena_bytes(shape: Shape, cap_groups: int, token_budget: Optional[int]) -> int:
    out = C.c_size_t(0)
    cs = shape.c()
    _check(load_library().stc_pass_host_arena_bytes(C.byref(cs), cap_groups,
                                                    -1 if token_budget is None else token_budget,
                                                    C.byref(out)), "stc_pass_host_arena_bytes")
    return int(out.value)


def pass_host(shape: Shape, k: torch.Tensor, v: torch.Tensor, scores: torch.Tensor,
              tok_class: Optional[torch.Tensor], q: torch.Tensor, token_budget: Optional[int],
              k_nominal: int, sm_scale: float, cap_groups: int, arena: torch.Tensor, out: torch.Tensor,
              total_groups: torch.Tensor, status: torch.Tensor, min_per_token: int = 1,
              mode: int = MODE_GLOBAL) -> None:
    """Whole pass from (pinned) host tensors; results land in host tensors after a stream sync."""
    cs = shape.c()
    _check(load_library().stc_pass_host(
        C.byref(cs), _hptr(k, torch.bfloat16, "k"), _hptr(v, torch.bfloat16, "v"),
        _hptr(scores, torch.float32, "scores"), _hptr(tok_class, torch.uint8, "tok_class"),
        _hptr(q, torch.bfloat16, "q"), -1 if token_budget is None else token_budget, k_nominal,
        min_per_token, mode, sm_scale, cap_groups, _ptr(arena, torch.uint8, "arena"), arena.numel(),
        _hptr(out, torch.float32, "out"), _hptr(total_groups, torch.int64, "total_groups"),
        _hptr(status, torch.int32, "status"), _stream()), "stc_pass_host")


def decode_step_host_arena_bytes(shape: Shape, token_budget: Optional[int]) -> int:
    out = C.c_size_t(0)
    cs = shape.c()
    _check(load_library().stc_decode_step_host_arena_bytes(
        C.byref(cs), -1 if token_budget is None else token_budget, C.byref(out)), "stc_decode_step_host_arena_bytes")
    return int(out.value)


def decode_step_host(shape: Shape, cache: Cache, q: torch.Tensor, token_budget: Optional[int], sm_scale: float,
                     arena: torch.Tensor, out: torch.Tensor, status: torch.Tensor) -> None:
    """One decode step (page selection + routed attention) on a device-resident cache, query and result in
    (pinned) host tensors; the results are valid after a stream sync."""
    cs, cc = shape.c(), cache.c()
    _check(load_library().stc_decode_step_host(
        C.byref(cs), C.byref(cc), _hptr(q, torch.bfloat16, "q"), -1 if token_budget is None else token_budget,
        sm_scale, _ptr(arena, torch.uint8, "arena"), arena.numel(), _hptr(out, torch.float32, "out"),
        _hptr(status, torch.int32, "status"), _stream()), "stc_decode_step_host")
