"""The two entry points that start from HOST buffers, against the CPU checker:
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
