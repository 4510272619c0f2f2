"""TEST INFRASTRUCTURE -- the CPU checker for the CUDA library.

Thin ctypes loader for ``stc_oracle.c`` (compiled with gcc on first use).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product package never does.

All functions take and return numpy arrays; bf16 tensors travel as uint16 bit
patterns (use :func:`bf16_bits` on a torch CPU tensor).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "stc_oracle.c"
_LIB = _HERE / "_build" / "libstc_oracle.so"

PAGE = 16
D = 128
MODE_GLOBAL, MODE_PER_TOKEN = 0, 1
CLS_DROP, CLS_ROUTED, CLS_FULL = 0, 1, 2


def build(force: bool = False) -> Path:
    """Compile the checker (plain C, no fast-math, no FMA contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call([
            "gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
            "-shared", "-fPIC", str(_SRC), "-o", str(tmp), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
        _lib.stc_o_bound_f32.restype = C.c_float
        _lib.stc_o_bound_f64.restype = C.c_double
        _lib.stc_o_select.restype = C.c_int32
        _lib.stc_o_route.restype = C.c_int32
        _lib.stc_o_pack.restype = C.c_int64
        _lib.stc_o_route_new_pages.restype = C.c_int64
        _lib.stc_o_kv_fraction.restype = C.c_double
        _lib.stc_o_max_threads.restype = C.c_int32
    return _lib


def bf16_bits(t) -> np.ndarray:
    """torch CPU bf16 tensor -> contiguous uint16 numpy array of its bits."""
    import torch
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32)


def _p(a, dtype=None):
    if a is None:
        return None
    if dtype is not None:
        assert a.dtype == dtype, (a.dtype, dtype)
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


def n_threads() -> int:
    return int(lib().stc_o_max_threads())


# ---------------------------------------------------------------- single problem
def page_meta(k: np.ndarray, length: int):
    """k uint16 [T,128] -> (kmin, kmax) uint16 [ceil(length/16),128]."""
    n_pages = (length + PAGE - 1) // PAGE
    kmin = np.zeros((n_pages, D), np.uint16)
    kmax = np.zeros((n_pages, D), np.uint16)
    lib().stc_o_page_meta(_p(np.ascontiguousarray(k), np.uint16), C.c_int32(length), _p(kmin), _p(kmax))
    return kmin, kmax


def bound_f32(q, kmin, kmax) -> float:
    return float(lib().stc_o_bound_f32(_p(np.ascontiguousarray(q), np.uint16),
                                       _p(np.ascontiguousarray(kmin), np.uint16),
                                       _p(np.ascontiguousarray(kmax), np.uint16)))


def bound_f64(q, kmin, kmax) -> float:
    return float(lib().stc_o_bound_f64(_p(np.ascontiguousarray(q), np.uint16),
                                       _p(np.ascontiguousarray(kmin), np.uint16),
                                       _p(np.ascontiguousarray(kmax), np.uint16)))


def page_scores(q_group, kmin, kmax) -> np.ndarray:
    """q_group uint16 [gq,128]; kmin/kmax uint16 [P,128] -> f32 [P]."""
    q_group = np.ascontiguousarray(q_group)
    u = np.zeros(kmin.shape[0], np.float32)
    lib().stc_o_page_scores(_p(q_group, np.uint16), C.c_int32(q_group.shape[0]),
                            _p(np.ascontiguousarray(kmin), np.uint16),
                            _p(np.ascontiguousarray(kmax), np.uint16),
                            C.c_int32(kmin.shape[0]), _p(u))
    return u


def select(u: np.ndarray, token_budget: int, n_recent_pages: int = 0) -> np.ndarray:
    u = np.ascontiguousarray(u, np.float32)
    ids = np.zeros(max(1, u.shape[0]), np.int32)
    k = lib().stc_o_select_recent(_p(u), C.c_int32(u.shape[0]), C.c_int32(token_budget),
                                  C.c_int32(n_recent_pages), _p(ids))
    return ids[:k].copy()


def route(scores: np.ndarray, cls, S: int, k_nominal: int, min_per_token: int = 1,
          mode: int = MODE_GLOBAL):
    """scores f32 [T,S]; cls uint8 [T] or None -> (rc, mask uint16 [T])."""
    scores = np.ascontiguousarray(scores, np.float32)
    T = scores.shape[0]
    mask = np.zeros(T, np.uint16)
    c = None if cls is None else np.ascontiguousarray(cls, np.uint8)
    rc = lib().stc_o_route(_p(scores), _p(c), C.c_int32(T), C.c_int32(S), C.c_int32(k_nominal),
                           C.c_int32(min_per_token), C.c_int32(mode), _p(mask))
    return int(rc), mask


def pack(v: np.ndarray, mask: np.ndarray, S: int, cap_groups: int):
    """v uint16 [T,128] -> (total, offs uint32 [T+1], packed uint16 [cap,128/S])."""
    T = v.shape[0]
    offs = np.zeros(T + 1, np.uint32)
    packed = np.zeros((max(cap_groups, 1), D // S), np.uint16)
    n = lib().stc_o_pack(_p(np.ascontiguousarray(v), np.uint16), _p(np.ascontiguousarray(mask), np.uint16),
                         C.c_int32(T), C.c_int32(S), C.c_int64(cap_groups), _p(offs), _p(packed))
    return int(n), offs, packed


def route_new_pages(scores, length, S, first_page, k_nominal, mask, offs, packed, min_per_token=1,
                    mode=MODE_GLOBAL):
    """In place on one problem: the complete pages from first_page on (stored at full width) are routed
    page by page, the open page's tokens move down.  scores f32 [T,S], mask u16 [T], offs u32 [T+1],
    packed u16 [cap,128/S].  Returns the new total (or -1 / -2, nothing changed)."""
    assert scores.dtype == np.float32 and mask.dtype == np.uint16 and offs.dtype == np.uint32
    assert packed.dtype == np.uint16
    for a in (scores, mask, offs, packed):
        assert a.flags["C_CONTIGUOUS"]
    return int(lib().stc_o_route_new_pages(_p(scores), C.c_int32(length), C.c_int32(S), C.c_int32(first_page),
                                           C.c_int32(k_nominal), C.c_int32(min_per_token), C.c_int32(mode),
                                           _p(mask), _p(offs), _p(packed)))


def attend_packed(q, k, packed, mask, offs, length, S, page_ids, scale):
    out = np.zeros(D, np.float64)
    lse = np.zeros(1, np.float64)
    ids = None if page_ids is None else np.ascontiguousarray(page_ids, np.int32)
    lib().stc_o_attend_packed(_p(np.ascontiguousarray(q), np.uint16), _p(np.ascontiguousarray(k), np.uint16),
                              _p(np.ascontiguousarray(packed), np.uint16),
                              _p(np.ascontiguousarray(mask), np.uint16),
                              _p(np.ascontiguousarray(offs), np.uint32), C.c_int32(length), C.c_int32(S),
                              _p(ids), C.c_int32(0 if ids is None else ids.shape[0]),
                              C.c_double(scale), _p(out), _p(lse))
    return out, float(lse[0])


def attend_masked_dense(q, k, v, mask, length, S, page_ids, scale):
    out = np.zeros(D, np.float64)
    lse = np.zeros(1, np.float64)
    ids = None if page_ids is None else np.ascontiguousarray(page_ids, np.int32)
    lib().stc_o_attend_masked_dense(_p(np.ascontiguousarray(q), np.uint16),
                                    _p(np.ascontiguousarray(k), np.uint16),
                                    _p(np.ascontiguousarray(v), np.uint16),
                                    _p(np.ascontiguousarray(mask), np.uint16), C.c_int32(length),
                                    C.c_int32(S), _p(ids),
                                    C.c_int32(0 if ids is None else ids.shape[0]),
                                    C.c_double(scale), _p(out), _p(lse))
    return out, float(lse[0])


def kv_fraction(n_tokens_original: int, n_tokens_retained: int, n_groups_kept: int, S: int) -> float:
    return float(lib().stc_o_kv_fraction(C.c_int64(n_tokens_original), C.c_int64(n_tokens_retained),
                                         C.c_int64(n_groups_kept), C.c_int32(S)))


# ---------------------------------------------------------------------- batched
def page_meta_batch(k, seq_len=None):
    """k uint16 [B,Hkv,T,128] -> kmin, kmax uint16 [B,Hkv,P,128]."""
    B, Hkv, T, _ = k.shape
    P = (T + PAGE - 1) // PAGE
    kmin = np.zeros((B, Hkv, P, D), np.uint16)
    kmax = np.zeros((B, Hkv, P, D), np.uint16)
    sl = None if seq_len is None else np.ascontiguousarray(seq_len, np.int32)
    lib().stc_o_page_meta_batch(C.c_int32(B), C.c_int32(Hkv), C.c_int32(T), _p(sl),
                                _p(np.ascontiguousarray(k), np.uint16), _p(kmin), _p(kmax))
    return kmin, kmax


def select_batch(q, kmin, kmax, token_budget, t_cap, seq_len=None, max_pages=None, want_scores=False,
                 n_recent_pages=0):
    """q uint16 [B,Hq,128] -> page_ids i32 [B,Hkv,max_pages], n_pages i32 [B,Hkv][, scores]."""
    B, Hq, _ = q.shape
    Hkv, P = kmin.shape[1], kmin.shape[2]
    if max_pages is None:
        max_pages = max(1, min(P, token_budget // PAGE))
    ids = np.full((B, Hkv, max_pages), -1, np.int32)
    n = np.zeros((B, Hkv), np.int32)
    sc = np.zeros((B, Hkv, P), np.float32) if want_scores else None
    sl = None if seq_len is None else np.ascontiguousarray(seq_len, np.int32)
    lib().stc_o_select_batch_recent(C.c_int32(B), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(t_cap), _p(sl),
                                    _p(np.ascontiguousarray(q), np.uint16), _p(np.ascontiguousarray(kmin), np.uint16),
                                    _p(np.ascontiguousarray(kmax), np.uint16), C.c_int32(token_budget),
                                    C.c_int32(n_recent_pages), C.c_int32(max_pages), _p(ids), _p(n), _p(sc))
    return (ids, n, sc) if want_scores else (ids, n)


def near_ties_batch(q, kmin, kmax, token_budget, t_cap, seq_len=None, rel=1e-6):
    """i32 [B,Hkv]: pages (other than the k-th itself) whose fp64 bound lies within
    rel*max(1,|U_k|) of the k-th largest bound of their problem."""
    B, Hq, _ = q.shape
    Hkv = kmin.shape[1]
    counts = np.zeros((B, Hkv), np.int32)
    sl = None if seq_len is None else np.ascontiguousarray(seq_len, np.int32)
    lib().stc_o_near_ties_batch(C.c_int32(B), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(t_cap), _p(sl),
                                _p(np.ascontiguousarray(q), np.uint16), _p(np.ascontiguousarray(kmin), np.uint16),
                                _p(np.ascontiguousarray(kmax), np.uint16), C.c_int32(token_budget),
                                C.c_double(rel), _p(counts))
    return counts


def route_pack_batch(v, scores, cls, S, k_nominal, cap_groups, seq_len=None, min_per_token=1,
                     mode=MODE_GLOBAL, cls_per_head=False):
    """v uint16 [B,Hkv,T,128]; scores f32 [B,Hkv,T,S]; cls uint8 [B,T] / [B,Hkv,T] / None."""
    B, Hkv, T, _ = v.shape
    mask = np.zeros((B, Hkv, T), np.uint16)
    offs = np.zeros((B, Hkv, T + 1), np.uint32)
    packed = np.zeros((B, Hkv, max(cap_groups, 1), D // S), np.uint16)
    total = np.zeros((B, Hkv), np.int64)
    status = np.zeros((B, Hkv), np.int32)
    sl = None if seq_len is None else np.ascontiguousarray(seq_len, np.int32)
    c = None if cls is None else np.ascontiguousarray(cls, np.uint8)
    lib().stc_o_route_pack_batch(C.c_int32(B), C.c_int32(Hkv), C.c_int32(T), _p(sl), C.c_int32(S),
                                 _p(np.ascontiguousarray(v), np.uint16),
                                 _p(np.ascontiguousarray(scores), np.float32), _p(c),
                                 C.c_int64(T if cls_per_head else 0), C.c_int32(k_nominal),
                                 C.c_int32(min_per_token), C.c_int32(mode), C.c_int64(cap_groups),
                                 _p(mask), _p(offs), _p(packed), _p(total), _p(status))
    return dict(mask=mask, offs=offs, packed=packed, total=total, status=status)


def attend_batch(q, k, S, mask, page_ids, n_pages, scale, packed=None, offs=None, v_dense=None,
                 seq_len=None):
    """out f64 [B,Hq,128], lse f64 [B,Hq]; reads the packed store unless v_dense is given."""
    B, Hq, _ = q.shape
    Hkv, T = k.shape[1], k.shape[2]
    out = np.zeros((B, Hq, D), np.float64)
    lse = np.zeros((B, Hq), np.float64)
    use_dense = 0 if v_dense is None else 1
    cap = 0 if packed is None else packed.shape[2]
    ids = None if page_ids is None else np.ascontiguousarray(page_ids, np.int32)
    npg = None if n_pages is None else np.ascontiguousarray(n_pages, np.int32)
    sl = None if seq_len is None else np.ascontiguousarray(seq_len, np.int32)
    lib().stc_o_attend_batch(C.c_int32(B), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(T), _p(sl),
                             C.c_int32(S), _p(np.ascontiguousarray(q), np.uint16),
                             _p(np.ascontiguousarray(k), np.uint16),
                             _p(None if v_dense is None else np.ascontiguousarray(v_dense), None),
                             _p(None if packed is None else np.ascontiguousarray(packed), None),
                             C.c_int64(cap), _p(np.ascontiguousarray(mask), np.uint16),
                             _p(None if offs is None else np.ascontiguousarray(offs), None),
                             _p(ids), _p(npg), C.c_int32(0 if ids is None else ids.shape[2]),
                             C.c_double(scale), C.c_int32(use_dense), _p(out), _p(lse))
    return out, lse


def router_logits(h, w, S, bias=None):
    """h uint16 [B,T,d_model], w uint16 [Hkv*S,d_model], bias f32 [B,Hkv*S] or None -> f64 [B,Hkv,T,S]."""
    B, T, dm = h.shape
    N = w.shape[0]
    Hkv = N // S
    out = np.zeros((B, Hkv, T, S), np.float64)
    b = None if bias is None else np.ascontiguousarray(bias, np.float32)
    lib().stc_o_router_logits(C.c_int32(B), C.c_int32(Hkv), C.c_int32(T), C.c_int32(S), C.c_int32(dm),
                              _p(np.ascontiguousarray(h), np.uint16), _p(np.ascontiguousarray(w), np.uint16),
                              _p(b), _p(out))
    return out


def query_bias(h_q, w_q, q_len=None):
    """h_q uint16 [B,Lq,d_model], w_q uint16 [N,d_model], q_len int32 [B] or None -> (s_q f64 [B,d_model], bias f64 [B,N])."""
    B, Lq, dm = h_q.shape
    N = w_q.shape[0]
    s_q = np.zeros((B, dm), np.float64)
    bias = np.zeros((B, N), np.float64)
    ql = None if q_len is None else np.ascontiguousarray(q_len, np.int32)
    lib().stc_o_query_bias(C.c_int32(B), C.c_int32(Lq), C.c_int32(dm), C.c_int32(N),
                           _p(np.ascontiguousarray(h_q), np.uint16), _p(ql),
                           _p(np.ascontiguousarray(w_q), np.uint16), _p(s_q), _p(bias))
    return s_q, bias


def pages_to_class(page_ids, n_pages, t_cap, seq_len=None):
    """Token classes of the paper's own stage order (Section 3.4 / Appendix B.1: the router sees the
    tokens Stage I retained): uint8 [B,Hkv,T], ROUTED for the valid tokens of the listed pages of each
    (batch, kv head) problem, DROP elsewhere.  Plain loops."""
    B, Hkv, _ = page_ids.shape
    cls = np.full((B, Hkv, t_cap), CLS_DROP, np.uint8)
    for b in range(B):
        length = t_cap if seq_len is None else int(seq_len[b])
        for h in range(Hkv):
            for i in range(int(n_pages[b, h])):
                p = int(page_ids[b, h, i])
                for t in range(p * PAGE, min((p + 1) * PAGE, length)):
                    if t >= 0:
                        cls[b, h, t] = CLS_ROUTED
    return cls
