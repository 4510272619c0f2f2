"""The two stages in the paper's own order (Section 3.4 / Appendix B.1: the value-group router acts
on the tokens Stage I retained, with the budget M = N*K over those N tokens): page selection first,
then routing + packing of the selected tokens only, then attention over the same pages.  It is the
same calls as the store-once order, linked by stc_pages_to_class; both orders run here on the
same inputs and each is held against the CPU checker run in that order."""
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


def run_paper_order(w, d, seq=None):
    B, Hkv, T, S = w.batch, w.n_kv_heads, w.t_cache, w.n_groups
    sl = d["seq_len"] if seq is None else torch.tensor(seq, dtype=torch.int32, device=DEV)
    shape = P.Shape(B, w.n_q_heads, Hkv, S, T, sl)
    cap = T * S
    cache = P.Cache.allocate(shape, d["k"], cap)
    cache.v_packed.fill_(float("nan"))
    P.build_page_meta(shape, cache)
    q = d["q"][0].contiguous()
    mp = max(1, min(shape.n_pages, w.token_budget // 16))
    ids = torch.full((B, Hkv, mp), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV)
    P.quest_select(shape, cache, q, w.token_budget, ids, npg, ws_s)
    cls = torch.full((B, Hkv, T), 0xEE, dtype=torch.uint8, device=DEV)
    P.pages_to_class(shape, ids, npg, cls)
    total = torch.full((B, Hkv), -7, dtype=torch.int64, device=DEV)
    status = torch.full((B, Hkv), -7, dtype=torch.int32, device=DEV)
    ws_r = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV)
    P.route_pack(shape, d["v"], d["scores"], cls, w.k_nominal, cache, total, status, ws_r)
    out = torch.full((B, w.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full((B, w.n_q_heads), float("nan"), dtype=torch.float32, device=DEV)
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, mp, device=DEV)
    P.decode_attn(shape, cache, q, ids, npg, H.SM_SCALE, out, ws_a, lse=lse)
    torch.cuda.synchronize()
    assert int(ws_a[:4].view(torch.int32)[0]) == 0

    # the checker, same order
    slc = sl.cpu().numpy()
    k, v, qb = H.cpu_bits(d["k"]), H.cpu_bits(d["v"]), H.cpu_bits(q)
    kmin, kmax = O.page_meta_batch(k, slc)
    ids_o, n_o = O.select_batch(qb, kmin, kmax, w.token_budget, T, slc)
    cls_o = O.pages_to_class(ids_o, n_o, T, slc)
    r = O.route_pack_batch(v, d["scores"].cpu().numpy(), cls_o, S, w.k_nominal, cap, slc, cls_per_head=True)
    out_o, lse_o = O.attend_batch(qb, k, S, r["mask"], ids_o, n_o, H.SM_SCALE, packed=r["packed"],
                                  offs=r["offs"], seq_len=slc)
    g = dict(cache=cache, total=total, status=status, page_ids=ids, n_pages=npg, out=out, lse=lse)
    o = dict(kmin=kmin, kmax=kmax, seq_len=slc, page_ids=ids_o, n_pages=n_o, out=out_o, lse=lse_o, **r)
    np.testing.assert_array_equal(cls.cpu().numpy(), cls_o)
    H.assert_bit_exact_write_side(w, g, o)
    H.assert_bit_exact_selection(g, o, check_scores=False)
    H.assert_attention_close(g, o)
    return g, o


def test_cfg0_both_orders():
    w = W.get("cfg0")
    d = W.make_inputs(w, DEV)
    g, o = run_paper_order(w, d)
    # budget over the selected tokens only: M = n_sel * K
    assert (o["total"] == 1024 * w.k_nominal).all()
    cnt = np.vectorize(lambda x: bin(int(x)).count("1"))(o["mask"])
    sel = O.pages_to_class(o["page_ids"], o["n_pages"], w.t_cache) == 1
    assert (cnt[sel] >= 1).all() and (cnt[~sel] == 0).all()
    # the store-once order on the same inputs (routing over all cached tokens) also matches its checker run,
    # and the two orders keep different group sets
    g2 = H.gpu_pipeline(w, d)
    o2 = H.oracle_pipeline(w, d)
    H.assert_bit_exact_write_side(w, g2, o2)
    H.assert_bit_exact_selection(g2, o2)
    H.assert_attention_close(g2, o2)
    np.testing.assert_array_equal(o2["page_ids"], o["page_ids"])
    assert (o2["mask"][sel] != o["mask"][sel]).any()


def test_grouped_heads_ragged_paper_order():
    w = W.shrink(W.get("cfg2"), batch=2, t_cache=16 * 90 + 5, token_budget=16 * 24)
    d = W.make_inputs(w, DEV)
    run_paper_order(w, d, seq=[16 * 90 + 5, 700])
