"""Page selection with Quest's local window (stc_quest_select_window): the most recent pages
are always kept and count against the budget; ids must equal the CPU checker's bit for bit,
for grouped and single query heads, ragged lengths, and windows from 0 to beyond the budget."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import workload as W

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("name,over,lens", [
    ("cfg0", dict(n_q_heads=4, n_kv_heads=4, batch=2, t_cache=16 * 200 + 7, token_budget=16 * 24), [3207, 1501]),
    ("cfg2", dict(batch=2, t_cache=16 * 700, token_budget=16 * 64), [11200, 16 * 65 + 1]),
])
@pytest.mark.parametrize("n_recent", [0, 4, 23, 24, 64, 1000])
def test_window_selection_matches_the_checker(name, over, lens, n_recent):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV)
    B, Hkv, T = w.batch, w.n_kv_heads, w.t_cache
    seq = torch.tensor(lens, dtype=torch.int32, device=DEV)
    shape = P.Shape(B, w.n_q_heads, Hkv, w.n_groups, T, seq)
    cache = P.Cache.allocate(shape, d["k"], 16)
    P.build_page_meta(shape, cache)
    max_pages = w.token_budget // 16
    ids = torch.full((B, Hkv, max_pages), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    u = torch.full((B, Hkv, shape.n_pages), float("nan"), dtype=torch.float32, device=DEV)
    q = d["q"][0].contiguous()
    P.quest_select(shape, cache, q, w.token_budget, ids, npg,
                   Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV), scores=u, n_recent_pages=n_recent)
    torch.cuda.synchronize()
    sl = seq.cpu().numpy()
    kmin, kmax = O.page_meta_batch(H.cpu_bits(d["k"]), sl)
    ids_o, n_o, u_o = O.select_batch(H.cpu_bits(q), kmin, kmax, w.token_budget, T, sl, want_scores=True,
                                     n_recent_pages=n_recent)
    g = dict(page_ids=ids, n_pages=npg, u=u)
    o = dict(page_ids=ids_o, n_pages=n_o, u=u_o, seq_len=sl)
    H.assert_bit_exact_selection(g, o)
    # the window really is in the list
    for b in range(B):
        np_b = (int(sl[b]) + 15) // 16
        k = min(max_pages, np_b)
        for hk in range(Hkv):
            row = ids[b, hk, :k].cpu().numpy()
            assert set(range(np_b - min(n_recent, k), np_b)) <= set(row.tolist())
