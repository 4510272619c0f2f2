"""The composed entry points against the CPU checker: stc_decode_step (selection + attention as one
device call) and the two that start from
HOST buffers:
stc_pass_host (the whole pass: copies in, metadata, routing + packing, selection, attention, copies
out) and stc_decode_step_host (one decode step on a device-resident cache: query in, selection +
attention, result out)."""
import numpy as np
import pytest
import torch

import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import workload as W

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"

CASES = [
    ("cfg0", dict(), None),
    ("cfg2", dict(batch=2, t_cache=16 * 140 + 3, token_budget=16 * 40), [16 * 140 + 3, 1777]),   # Gq = 7, ragged
    ("cfg4", dict(batch=2, n_q_heads=8, n_kv_heads=2, t_cache=16 * 300 + 1, token_budget=1024), None),
    ("cfg3", dict(batch=3, n_q_heads=4, n_kv_heads=4), None),                                     # classes, selection off
]


def pinned(t):
    return t.cpu().contiguous().pin_memory()


@pytest.mark.parametrize("name,over,seq", CASES)
def test_pass_host_matches_the_checker(name, over, seq):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV)
    sl = d["seq_len"] if seq is None else torch.tensor(seq, dtype=torch.int32, device=DEV)
    shape = P.Shape(w.batch, w.n_q_heads, w.n_kv_heads, w.n_groups, w.t_cache, sl)
    cap = w.t_cache * w.n_groups
    o = H.oracle_pipeline(w, d, seq_len=None if seq is None else seq)
    hk, hv, hs = pinned(d["k"]), pinned(d["v"]), pinned(d["scores"])
    hc = None if d["tok_class"] is None else pinned(d["tok_class"])
    hq = pinned(d["q"][0])
    h_out = torch.full((w.batch, w.n_q_heads, 128), float("nan")).pin_memory()
    h_tot = torch.full((w.batch, w.n_kv_heads), -7, dtype=torch.int64).pin_memory()
    h_st = torch.full((w.batch, w.n_kv_heads), -7, dtype=torch.int32).pin_memory()
    arena = torch.empty(Bd.pass_host_arena_bytes(shape, cap, w.token_budget), dtype=torch.uint8, device=DEV)
    arena.fill_(0xA5)
    for _ in range(2):                                       # the arena is reusable by the next call
        Bd.pass_host(shape, hk, hv, hs, hc, hq, w.token_budget, w.k_nominal, H.SM_SCALE, cap, arena,
                     h_out, h_tot, h_st)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(h_tot.numpy(), o["total"])
        assert (h_st.numpy() == 0).all() and (o["status"] == 0).all()
        max_abs, mean_rel = H.attn_errors(h_out, o["out"])
        assert max_abs <= H.MAX_ABS_TOL and mean_rel <= H.MEAN_REL_TOL, (max_abs, mean_rel)


@pytest.mark.parametrize("name,over,seq", CASES)
def test_decode_step_host_matches_the_checker(name, over, seq):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV, n_queries=2)
    g = H.gpu_pipeline(w, d, seq_len=seq)                    # builds the device-resident cache
    shape, cache = g["shape"], g["cache"]
    arena = torch.empty(Bd.decode_step_host_arena_bytes(shape, w.token_budget), dtype=torch.uint8, device=DEV)
    arena.fill_(0x5A)
    h_out = torch.full((w.batch, w.n_q_heads, 128), float("nan")).pin_memory()
    h_st = torch.full((1,), -7, dtype=torch.int32).pin_memory()
    for qi in (1, 0):
        o = H.oracle_pipeline(w, d, seq_len=seq, q_index=qi)
        Bd.decode_step_host(shape, cache, pinned(d["q"][qi]), w.token_budget, H.SM_SCALE, arena, h_out, h_st)
        torch.cuda.synchronize()
        assert int(h_st[0]) == 0
        max_abs, mean_rel = H.attn_errors(h_out, o["out"])
        assert max_abs <= H.MAX_ABS_TOL and mean_rel <= H.MEAN_REL_TOL, (max_abs, mean_rel)


@pytest.mark.parametrize("name,over,seq", CASES[:3] + [("cfg4", dict(batch=2, t_cache=16 * 4200 + 3), None)])
def test_decode_step_equals_the_two_calls_and_the_checker(name, over, seq):
    """Eager and replayed from a CUDA graph."""
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV, n_queries=3)
    g = H.gpu_pipeline(w, d, seq_len=seq, want_scores=False)          # select, then attend: two calls
    shape, cache = g["shape"], g["cache"]
    B, Hkv, Hq = w.batch, w.n_kv_heads, w.n_q_heads
    mp = g["page_ids"].shape[-1]
    ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV); ws_s.fill_(0x11)
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, mp, device=DEV); ws_a.fill_(0x22)
    ids = torch.full((B, Hkv, mp), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    q0 = d["q"][0].contiguous()
    P.decode_step(shape, cache, q0, w.token_budget, ids, npg, H.SM_SCALE, out, ws_s, ws_a, lse=lse)
    torch.cuda.synchronize()
    assert int(ws_a[:4].view(torch.int32)[0]) == 0 and int(ws_s[:4].view(torch.int32)[0]) == 0
    assert torch.equal(ids, g["page_ids"]) and torch.equal(npg, g["n_pages"])
    assert torch.equal(out, g["out"]) and torch.equal(lse, g["lse"])      # the same kernels: bit for bit
    o = H.oracle_pipeline(w, d, seq_len=seq)
    H.assert_bit_exact_selection(dict(page_ids=ids, n_pages=npg), o, check_scores=False)
    H.assert_attention_close(dict(out=out, lse=lse), o)
    # captured once per query, replayed out of order
    qs = [d["q"][i].contiguous() for i in range(3)]
    graphs = []
    for i in range(3):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            P.decode_step(shape, cache, qs[i], w.token_budget, ids, npg, H.SM_SCALE, out, ws_s, ws_a, lse=lse)
        graphs.append(gr)
    for i in (2, 0, 1, 1, 2):
        graphs[i].replay()
    torch.cuda.synchronize()
    o2 = H.oracle_pipeline(w, d, seq_len=seq, q_index=2)
    H.assert_bit_exact_selection(dict(page_ids=ids, n_pages=npg), o2, check_scores=False)
    H.assert_attention_close(dict(out=out, lse=lse), o2)
