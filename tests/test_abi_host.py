"""Host-only checks of the C-ABI library: it loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import re
from pathlib import Path

import pytest

import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import build as B

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.load_library()


def declared_symbols():
    names = set()
    for h in (ROOT / "include").glob("*.h"):
        names |= set(re.findall(r"\b(stc_[a-z_0-9]+)\s*\(", h.read_text()))
    return names


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert set(Bd.EXPORTS) <= names and len(names) >= 8
    for n in names:
        assert hasattr(lib, n), n
    assert lib.stc_version() >= 100
    assert lib.stc_status_string(0) == b"ok"
    assert b"workspace" in lib.stc_status_string(3)


def shape(**kw):
    base = dict(batch=1, n_q_heads=8, n_kv_heads=8, n_groups=8, t_cap=4096)
    base.update(kw)
    return P.Shape(**base)


def test_workspace_sizes_and_shape_validation(lib):
    s = shape()
    for op in (Bd.OP_QUEST_SELECT, Bd.OP_ROUTE_PACK, Bd.OP_DECODE_ATTN):
        n = P.workspace_bytes(s, op, 64)
        assert n > 0 and n % 256 == 0
    assert P.workspace_bytes(shape(batch=0), Bd.OP_ROUTE_PACK) == 0
    for bad, code in [(dict(head_dim=64), 2), (dict(page_size=32), 2), (dict(n_groups=5), 2),
                      (dict(n_q_heads=9), 1), (dict(n_q_heads=72), 2), (dict(t_cap=-1), 1),
                      (dict(t_cap=1 << 28), 2)]:
        with pytest.raises(P.StcError) as e:
            P.workspace_bytes(shape(**bad), Bd.OP_QUEST_SELECT)
        assert e.value.code == code, bad
    with pytest.raises(P.StcError):
        P.workspace_bytes(s, 99)


def test_calls_reject_bad_arguments_before_any_launch(lib):
    cs = shape().c()
    cc = Bd._Cache()                      # all null
    st = None
    assert lib.stc_build_page_meta(C.byref(cs), C.byref(cc), 0, -1, st) == 1
    assert lib.stc_build_page_meta(None, C.byref(cc), 0, -1, st) == 1
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), None, 1024, 64, None, None, None, None, 0, st) == 1
    assert lib.stc_route_pack(C.byref(cs), None, None, None, 0, 4, 1, 0, C.byref(cc), None, None, None, 0, st) == 1
    assert lib.stc_route_pack(C.byref(cs), None, None, None, 0, 9, 1, 0, C.byref(cc), None, None, None, 0, st) == 1
    assert lib.stc_route_pack(C.byref(cs), None, None, None, 17, 4, 1, 0, C.byref(cc), None, None, None, 0, st) == 1
    assert lib.stc_decode_attn(C.byref(cs), C.byref(cc), None, None, None, 0, 0.1, None, None, None, 0, st) == 1
    # non-null fakes (never dereferenced on the host) reach the workspace checks
    fake = C.c_void_p(0x1000)
    cc = Bd._Cache(fake, fake, fake, fake, fake, fake, 100)
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), fake, 1024, 63, fake, fake, None, fake, 1 << 30, st) == 1
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), fake, 1024, 64, fake, fake, None, None, 0, st) == 3
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), fake, 1024, 64, fake, fake, None, C.c_void_p(0x1010), 1 << 30, st) == 3
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), fake, 1024, 64, fake, fake, None, fake, 16, st) == 3
    assert lib.stc_decode_attn(C.byref(cs), C.byref(cc), fake, fake, None, 64, 0.1, fake, None, fake, 1 << 30, st) == 1
    assert lib.stc_decode_attn(C.byref(cs), C.byref(cc), fake, fake, fake, 64, 0.1, fake, None, fake, 16, st) == 3
    # tensors the kernels move in 16-byte pieces must start on 16-byte boundaries
    odd = C.c_void_p(0x1008)
    assert lib.stc_quest_select(C.byref(cs), C.byref(cc), odd, 1024, 64, fake, fake, None, fake, 1 << 30, st) == 1
    assert lib.stc_decode_attn(C.byref(cs), C.byref(cc), odd, fake, fake, 64, 0.1, fake, None, fake, 1 << 30, st) == 1
    assert lib.stc_decode_attn(C.byref(cs), C.byref(cc), fake, fake, fake, 64, 0.1, odd, None, fake, 1 << 30, st) == 1
    assert lib.stc_route_pack(C.byref(cs), fake, odd, None, 0, 4, 1, 0, C.byref(cc), fake, fake, fake, 1 << 30, st) == 1
    assert lib.stc_route_pack(C.byref(cs), odd, fake, None, 0, 4, 1, 0, C.byref(cc), fake, fake, fake, 1 << 30, st) == 1
    cc_odd = Bd._Cache(odd, fake, fake, fake, fake, fake, 100)
    assert lib.stc_build_page_meta(C.byref(cs), C.byref(cc_odd), 0, -1, st) == 1
    # the window variant: a negative window is an argument error, a valid one reaches the workspace check
    assert lib.stc_quest_select_window(C.byref(cs), C.byref(cc), fake, 1024, -1, 64, fake, fake, None, fake, 1 << 30, st) == 1
    assert lib.stc_quest_select_window(C.byref(cs), C.byref(cc), fake, 1024, 4, 64, fake, fake, None, None, 0, st) == 3
    # query summary: sizes, alignment and the multiple-of-8 rule are checked on the host
    assert lib.stc_query_bias(-1, 4, 64, 16, fake, None, fake, fake, fake, st) == 1
    assert lib.stc_query_bias(2, 4, 0, 16, fake, None, fake, fake, fake, st) == 1
    assert lib.stc_query_bias(2, 4, 60, 16, fake, None, fake, fake, fake, st) == 2
    assert lib.stc_query_bias(2, 4, 64, 16, C.c_void_p(0x1008), None, fake, fake, fake, st) == 1
    assert lib.stc_query_bias(2, 4, 64, 16, fake, None, fake, None, fake, st) == 1
    assert lib.stc_query_bias(0, 4, 64, 16, None, None, None, None, None, st) == 0


def test_cache_bytes_reproduces_the_closed_form(lib):
    # r = 1/4 of 2048 tokens, K/S = 2/8: (512*256 + 1024*32) / (2048*512) = 15.625 %
    kv, idx = P.cache_bytes(512, 1024, 8)
    assert kv / (2048 * 512) == 0.15625
    assert idx == 512 * 2 + 513 * 4 + 32 * 512
    kv, _ = P.cache_bytes(256, 256 * 7, 8)                 # r = 1/8, K/S = 7/8
    assert kv / (2048 * 512) == 0.1171875


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(Bd, "_lib", None)
    monkeypatch.setattr(Bd, "_LIB_PATH", tmp_path / "libstc.so")
    with pytest.raises(ImportError):
        Bd.load_library()


def test_newer_calls_reject_bad_arguments_before_any_launch(lib):
    cs = shape().c()
    cc = Bd._Cache()
    st = None
    fake = C.c_void_p(0x1000)
    full = Bd._Cache(fake, fake, fake, fake, fake, fake, 100)
    # stc_decode_step: null cache pointers, list stride below the budget's page count, workspaces missing
    assert lib.stc_decode_step(C.byref(cs), C.byref(cc), fake, 1024, 64, fake, fake, 0.1, fake, None, fake, 1 << 30,
                               fake, 1 << 30, st) == 1
    assert lib.stc_decode_step(C.byref(cs), C.byref(full), fake, 1024, 63, fake, fake, 0.1, fake, None, fake, 1 << 30,
                               fake, 1 << 30, st) == 1
    assert lib.stc_decode_step(C.byref(cs), C.byref(full), fake, 1024, 64, fake, fake, 0.1, fake, None, None, 0,
                               fake, 1 << 30, st) == 3
    assert lib.stc_decode_step(C.byref(cs), C.byref(full), fake, 1024, 64, fake, fake, 0.1, fake, None, fake, 1 << 30,
                               fake, 16, st) == 3
    # stc_route_new_pages: budget above S, bad mode, null scores
    assert lib.stc_route_new_pages(C.byref(cs), C.byref(full), fake, fake, 9, 1, 0, fake, fake, st) == 1
    assert lib.stc_route_new_pages(C.byref(cs), C.byref(full), fake, fake, 4, 1, 7, fake, fake, st) == 1
    assert lib.stc_route_new_pages(C.byref(cs), C.byref(full), None, fake, 4, 1, 0, fake, fake, st) == 1
    # stc_pages_to_class: null output
    assert lib.stc_pages_to_class(C.byref(cs), fake, fake, 64, None, st) == 1
    # stc_decode_step_host: arena too small
    out = C.c_size_t(0)
    assert lib.stc_decode_step_host_arena_bytes(C.byref(cs), 1024, C.byref(out)) == 0 and out.value > 0
    assert lib.stc_decode_step_host(C.byref(cs), C.byref(full), fake, 1024, 0.1, fake, 16, fake, fake, st) == 3
