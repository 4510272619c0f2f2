"""Streaming append (stc_append_tokens): a decode loop that grows the cache one token at a
time must end in exactly the state the CPU checker reaches when it routes the original
tokens and keeps the appended ones at full width (Section 3.4 leaves the query region uncompressed),
and attention over that state must agree with the checker."""
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


@pytest.mark.parametrize("name,over", [("cfg2", dict(batch=2, t_cache=16 * 60, token_budget=16 * 12)),
                                       ("cfg0", dict(n_q_heads=2, n_kv_heads=2, batch=2, t_cache=16 * 60 + 5,
                                                     token_budget=16 * 9))])
def test_decode_loop_with_appends_matches_the_checker(name, over):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV, n_queries=2)
    B, Hkv, T, S = w.batch, w.n_kv_heads, w.t_cache, w.n_groups
    old = [500, 333]
    cur = torch.tensor(old, dtype=torch.int32, device=DEV)
    shape = P.Shape(B, w.n_q_heads, Hkv, S, T, cur)
    cache = P.Cache.allocate(shape, d["k"], T * S)
    cache.v_packed.fill_(float("nan")); cache.kmin.fill_(float("nan")); cache.kmax.fill_(float("nan"))
    total = torch.zeros(B, Hkv, dtype=torch.int64, device=DEV)
    status = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    P.build_page_meta(shape, cache)
    ws = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV)
    P.route_pack(shape, d["v"], d["scores"], None, w.k_nominal, cache, total, status, ws)

    # 17 single-token steps (both sequences cross a page boundary), then 5 tokens at once
    for n_new in [1] * 17 + [5]:
        old_len = cur.clone()
        cur += n_new                                   # shape.seq_len is this tensor: lengths after the append
        P.append_tokens(shape, cache, d["v"], old_len, n_new, total, status)
    torch.cuda.synchronize()
    final = [x + 22 for x in old]
    assert cur.tolist() == final and (status == 0).all()

    # checker: original tokens routed, appended tokens full width, metadata over the final lengths
    cls = np.zeros((B, T), np.uint8)
    for b in range(B):
        cls[b, :old[b]] = O.CLS_ROUTED
        cls[b, old[b]:final[b]] = O.CLS_FULL
    sl = np.asarray(final, np.int32)
    k_bits, v_bits = H.cpu_bits(d["k"]), H.cpu_bits(d["v"])
    r = O.route_pack_batch(v_bits, d["scores"].cpu().numpy(), cls, S, w.k_nominal, T * S, sl)
    kmin, kmax = O.page_meta_batch(k_bits, sl)
    o = dict(kmin=kmin, kmax=kmax, seq_len=sl, **r)
    H.assert_bit_exact_write_side(w, dict(cache=cache, total=total, status=status), o)
    assert (r["total"] == np.array(old)[:, None] * w.k_nominal + 22 * S).all()

    # read side on the grown cache
    q = d["q"][1].contiguous()
    max_pages = w.token_budget // 16
    ids = torch.full((B, Hkv, max_pages), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    u = torch.full((B, Hkv, shape.n_pages), float("nan"), dtype=torch.float32, device=DEV)
    P.quest_select(shape, cache, q, w.token_budget, ids, npg, Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV),
                   scores=u)
    out = torch.zeros(B, w.n_q_heads, 128, dtype=torch.float32, device=DEV)
    lse = torch.zeros(B, w.n_q_heads, dtype=torch.float32, device=DEV)
    P.decode_attn(shape, cache, q, ids, npg, H.SM_SCALE, out,
                  Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, max_pages, device=DEV), lse=lse)
    torch.cuda.synchronize()
    qb = H.cpu_bits(q)
    ids_o, n_o, u_o = O.select_batch(qb, kmin, kmax, w.token_budget, T, sl, want_scores=True)
    out_o, lse_o = O.attend_batch(qb, k_bits, S, r["mask"], ids_o, n_o, H.SM_SCALE, packed=r["packed"],
                                  offs=r["offs"], seq_len=sl)
    g = dict(page_ids=ids, n_pages=npg, u=u, out=out, lse=lse)
    oo = dict(page_ids=ids_o, n_pages=n_o, u=u_o, out=out_o, lse=lse_o, seq_len=sl)
    H.assert_bit_exact_selection(g, oo)
    H.assert_attention_close(g, oo)


def test_inconsistent_lengths_are_reported_and_leave_the_cache_alone():
    w = W.shrink(W.get("cfg0"), n_q_heads=2, n_kv_heads=2, batch=2, t_cache=400)
    d = W.make_inputs(w, DEV)
    cur = torch.tensor([100, 200], dtype=torch.int32, device=DEV)
    shape = P.Shape(2, 2, 2, w.n_groups, 400, cur)
    cache = P.Cache.allocate(shape, d["k"], 400 * 8)
    total = torch.zeros(2, 2, dtype=torch.int64, device=DEV)
    status = torch.zeros(2, 2, dtype=torch.int32, device=DEV)
    P.build_page_meta(shape, cache)
    P.route_pack(shape, d["v"], d["scores"], None, 4, cache, total, status,
                 Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV))
    before = (cache.v_mask.clone(), cache.v_offs.clone(), total.clone())
    old_len = torch.tensor([120, 190], dtype=torch.int32, device=DEV)   # seq 0 "shrinks", seq 1 adds 10 > max_new
    P.append_tokens(shape, cache, d["v"], old_len, 4, total, status)
    torch.cuda.synchronize()
    assert (status == 1).all()
    assert torch.equal(cache.v_mask, before[0]) and torch.equal(cache.v_offs, before[1])
