"""Page selection without a score output, several query heads per KV head: the tensor-core scan
scores the pages approximately, and only the pages within a rigorous margin of the k-th score are
re-scored in the declared fp32 order.  The page ids must still be those of the CPU checker, bit for
bit, on ordinary inputs, with exact ties (duplicated pages), with hosts of near-ties, when every
page ties (the scan then falls back to scoring everything exactly), with the local window, ragged
lengths and rows too long to stage in shared memory."""
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


def select_both_ways(w, d, seq=None, budget=None, n_recent=0, q_index=0, want_ws=False):
    B, Hkv, T = w.batch, w.n_kv_heads, w.t_cache
    sl = d["seq_len"] if seq is None else torch.tensor(seq, dtype=torch.int32, device=DEV)
    shape = P.Shape(B, w.n_q_heads, Hkv, w.n_groups, T, sl)
    cache = P.Cache.allocate(shape, d["k"], 1)
    P.build_page_meta(shape, cache)
    bud = w.token_budget if budget is None else budget
    mp = max(1, min(shape.n_pages, bud // 16))
    q = d["q"][q_index].contiguous()
    ws = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV)
    ws.fill_(0xCD)
    ids = torch.full((B, Hkv, mp), -1, dtype=torch.int32, device=DEV)
    n = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    P.quest_select(shape, cache, q, bud, ids, n, ws, n_recent_pages=n_recent)          # no scores: filtered scan
    torch.cuda.synchronize()
    ws_after = ws.clone() if want_ws else None
    ids_x = torch.full_like(ids, -1); n_x = torch.full_like(n, -1)
    u = torch.full((B, Hkv, shape.n_pages), float("nan"), dtype=torch.float32, device=DEV)
    P.quest_select(shape, cache, q, bud, ids_x, n_x, ws, scores=u, n_recent_pages=n_recent)   # exact scan
    torch.cuda.synchronize()
    slc = sl.cpu().numpy()
    ids_o, n_o, u_o = O.select_batch(H.cpu_bits(q), H.cpu_bits(cache.kmin), H.cpu_bits(cache.kmax), bud, T, slc,
                                     want_scores=True, n_recent_pages=n_recent)
    np.testing.assert_array_equal(n.cpu().numpy(), n_o)
    np.testing.assert_array_equal(n_x.cpu().numpy(), n_o)
    ids_g, ids_gx = ids.cpu().numpy(), ids_x.cpu().numpy()
    for b in range(B):
        for h in range(Hkv):
            k = int(n_o[b, h])
            np.testing.assert_array_equal(ids_g[b, h, :k], ids_o[b, h, :k], err_msg=f"filtered scan, problem {(b, h)}")
            np.testing.assert_array_equal(ids_gx[b, h, :k], ids_o[b, h, :k], err_msg=f"exact scan, problem {(b, h)}")
            assert (ids_g[b, h, k:] == -1).all()
    return dict(shape=shape, cache=cache, ws=ws_after, u_exact=u, u_o=u_o, n_o=n_o, seq=slc)


@pytest.mark.parametrize("gq", [2, 3, 4, 5, 7, 8])
def test_filtered_selection_matches_the_checker(gq):
    w = W.shrink(W.get("cfg4"), batch=3, n_q_heads=2 * gq, n_kv_heads=2, t_cache=16 * 4234 + 7, token_budget=16 * 150)
    d = W.make_inputs(w, DEV, n_queries=2)
    for qi in range(2):
        select_both_ways(w, d, seq=[w.t_cache, 16 * 517 + 1, 16 * 128], q_index=qi)


@pytest.mark.parametrize("budget", [16, 48, 16 * 700, 16 * 4233])
def test_budget_extremes(budget):
    w = W.shrink(W.get("cfg4"), batch=2, n_q_heads=8, n_kv_heads=2, t_cache=16 * 4234 + 7)
    d = W.make_inputs(w, DEV)
    select_both_ways(w, d, budget=budget)


def test_exact_ties_between_duplicated_pages_go_to_the_lower_page():
    w = W.shrink(W.get("cfg4"), batch=1, n_q_heads=8, n_kv_heads=2, t_cache=16 * 4512, token_budget=16 * 61)
    d = W.make_inputs(w, DEV)
    k = d["k"].view(1, 2, 4512, 16, 128)
    k[:, :, 1::2] = k[:, :, 0::2].clone()                  # every page has an identical twin
    r = select_both_ways(w, d)
    assert H.near_tie_pages(r["u_o"][0, 0], 61) >= 1


def test_every_page_identical_takes_the_exact_fallback():
    # 5000 identical pages: all of them lie inside the margin, far more than the list of pages to settle holds
    w = W.shrink(W.get("cfg4"), batch=1, n_q_heads=8, n_kv_heads=2, t_cache=16 * 5000, token_budget=16 * 100)
    d = W.make_inputs(w, DEV)
    k = d["k"].view(1, 2, 5000, 16, 128)
    k[:] = k[:, :, :1].clone()
    r = select_both_ways(w, d)
    assert (r["n_o"] == 100).all()


def test_a_crowd_of_near_ties_around_the_threshold():
    # pages 200..1199 are copies of one page with the lowest mantissa bit of ONE key element flipped here and
    # there: their bounds differ by a few ulps, hundreds of them straddle the threshold
    w = W.shrink(W.get("cfg4"), batch=1, n_q_heads=4, n_kv_heads=1, t_cache=16 * 4200, token_budget=16 * 700)
    d = W.make_inputs(w, DEV)
    k = d["k"].view(1, 1, 4200, 16, 128)
    k[:, :, 200:1200] = k[:, :, 200:201].clone()
    kb = d["k"].view(torch.int16).view(1, 1, 4200, 16, 128)
    g = torch.Generator(device="cpu"); g.manual_seed(5)
    for p in range(200, 1200):
        t, c = int(torch.randint(0, 16, (1,), generator=g)), int(torch.randint(0, 128, (1,), generator=g))
        kb[0, 0, p, t, c] ^= 1
    select_both_ways(w, d)


@pytest.mark.parametrize("n_recent", [1, 4, 40])
def test_local_window_with_the_filtered_scan(n_recent):
    w = W.shrink(W.get("cfg2"), batch=2, t_cache=16 * 1300 + 9, token_budget=16 * 30)     # Gq = 7
    d = W.make_inputs(w, DEV)
    select_both_ways(w, d, seq=[16 * 1300 + 9, 16 * 37 + 2], n_recent=n_recent)


def test_rows_too_long_to_stage_in_shared_memory():
    w = W.shrink(W.get("cfg4"), batch=1, n_q_heads=4, n_kv_heads=1, t_cache=16 * 20000 + 3, token_budget=16 * 900)
    d = W.make_inputs(w, DEV)
    select_both_ways(w, d)


def test_many_short_problems_and_empty_sequences():
    # capacity of 1100 pages per sequence (Gq = 7), most sequences far shorter
    w = W.shrink(W.get("cfg2"), batch=50, n_q_heads=14, n_kv_heads=2, t_cache=16 * 1100 + 5, token_budget=16 * 9)
    d = W.make_inputs(w, DEV)
    g0 = torch.Generator(device="cpu"); g0.manual_seed(3)
    seq = torch.randint(0, 16 * 60, (50,), generator=g0).tolist()
    seq[0] = 0; seq[1] = 1; seq[2] = w.t_cache; seq[3] = 16 * 9; seq[4] = 16 * 9 + 1; seq[5] = 16 * 700 + 3
    select_both_ways(w, d, seq=seq)


def test_the_margin_of_the_filter_has_room_to_spare():
    """The approximate scores left in the workspace (layout: a 256-byte block with the status word, four
    words per problem -- arrival counters [problems], largest sum|term| [problems], two key bounds -- padded
    to 256 bytes, then f32 [problems][P]) against the declared-order scores: the difference must stay below
    an eighth of the margin the kernel allows itself."""
    w = W.shrink(W.get("cfg4"), batch=2, n_q_heads=16, n_kv_heads=2, t_cache=16 * 4100, token_budget=16 * 200)
    d = W.make_inputs(w, DEV)
    r = select_both_ways(w, d, want_ws=True)
    problems, Pn = 4, r["shape"].n_pages
    ws = r["ws"]
    assert int(ws[:4].view(torch.int32)[0]) == 0                         # device status word
    absmax = ws[256 + problems * 4: 256 + problems * 8].view(torch.float32).cpu().numpy()
    off = 256 + (problems * 16 + 255) // 256 * 256
    approx = ws[off: off + problems * Pn * 4].view(torch.float32).view(problems, Pn).cpu().numpy()
    exact = r["u_o"].reshape(problems, Pn)
    for p in range(problems):
        delta = absmax[p] * 1.01 / 8192.0
        fin = np.isfinite(approx[p])                       # pages settled exactly may carry marks
        err = np.abs(approx[p][fin].astype(np.float64) - exact[p][fin]).max()
        assert absmax[p] > 0 and err <= delta / 8, (p, err, delta)
