"""Parity at the benchmarked sizes: every (batch, kv head) problem of every configuration against
the CPU checker -- page metadata, masks, offsets, packed store, totals, page ids and the fp32 score
bits bit for bit, attention within the stated tolerance.

cfg1 and cfg2 run whole in one piece.  cfg4 (8 GiB of keys and values) runs whole on the GPU and is
checked one sequence at a time so the checker's host copies stay small; its 12 sweep points
(token budget x kept groups) run at the full 131072-token context, the write side once per
keep ratio, selection and attention per budget."""
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


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_whole_config_every_problem(name):
    w = W.get(name)
    d = W.make_inputs(w, DEV)
    g = H.gpu_pipeline(w, d, cap_groups=w.t_cache * w.k_nominal)
    o = H.oracle_pipeline(w, d, cap_groups=w.t_cache * w.k_nominal)
    H.assert_bit_exact_write_side(w, g, o)
    H.assert_bit_exact_selection(g, o)
    H.assert_attention_close(g, o)
    assert (o["n_pages"] == w.token_budget // 16).all()
    assert (o["total"] == w.t_cache * w.k_nominal).all()


class Cfg4:
    """cfg4 inputs on the device plus, per sequence, the checker's view of them."""

    def __init__(self):
        self.w = W.get("cfg4")
        w = self.w
        self.d = W.make_inputs(w, DEV, n_queries=2)
        self.shape = P.Shape(w.batch, w.n_q_heads, w.n_kv_heads, w.n_groups, w.t_cache, self.d["seq_len"])
        self.w1 = W.shrink(w, batch=1)

    def cpu_sequence(self, b):
        d = self.d
        return dict(k=H.cpu_bits(d["k"][b:b + 1]), v=H.cpu_bits(d["v"][b:b + 1]),
                    scores=d["scores"][b:b + 1].cpu().numpy(),
                    seq_len=d["seq_len"][b:b + 1].cpu().numpy())


@pytest.fixture(scope="module")
def cfg4():
    c = Cfg4()
    yield c
    del c
    torch.cuda.empty_cache()


def _write_side_gpu(c, keep):
    w, d, shape = c.w, c.d, c.shape
    cap = w.t_cache * keep
    cache = P.Cache.allocate(shape, d["k"], cap)
    cache.kmin.fill_(float("nan")); cache.kmax.fill_(float("nan")); cache.v_packed.fill_(float("nan"))
    P.build_page_meta(shape, cache)
    total = torch.full((w.batch, w.n_kv_heads), -7, dtype=torch.int64, device=DEV)
    status = torch.full((w.batch, w.n_kv_heads), -7, dtype=torch.int32, device=DEV)
    ws = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV)
    ws.fill_(0xAB)
    P.route_pack(shape, d["v"], d["scores"], None, keep, cache, total, status, ws)
    torch.cuda.synchronize()
    return cache, total, status, cap


def _read_side_gpu(c, cache, budget, q):
    w, shape = c.w, c.shape
    mp = budget // 16
    ids = torch.full((w.batch, w.n_kv_heads, mp), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((w.batch, w.n_kv_heads), -1, dtype=torch.int32, device=DEV)
    u = torch.full((w.batch, w.n_kv_heads, shape.n_pages), float("nan"), dtype=torch.float32, device=DEV)
    ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV); ws_s.fill_(0xCD)
    P.quest_select(shape, cache, q, budget, ids, npg, ws_s, scores=u)
    # the same selection without the score output (the benchmark's call): ids must not depend on it
    ids2, npg2 = torch.full_like(ids, -1), torch.full_like(npg, -1)
    P.quest_select(shape, cache, q, budget, ids2, npg2, ws_s)
    out = torch.full((w.batch, w.n_q_heads, 128), float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full((w.batch, w.n_q_heads), float("nan"), dtype=torch.float32, device=DEV)
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, mp, device=DEV); ws_a.fill_(0xEF)
    P.decode_attn(shape, cache, q, ids, npg, H.SM_SCALE, out, ws_a, lse=lse)
    torch.cuda.synchronize()
    assert int(ws_a[:4].view(torch.int32)[0]) == 0
    assert torch.equal(ids, ids2) and torch.equal(npg, npg2)
    return dict(page_ids=ids, n_pages=npg, u=u, out=out, lse=lse)


def _slice_b(t, b):
    return t[b:b + 1]


@pytest.mark.parametrize("keep", W.CFG4_KEEPS)
def test_cfg4_every_problem_and_every_sweep_point_at_full_context(cfg4, keep):
    c = cfg4
    w, d = c.w, c.d
    S = w.n_groups
    cache, total, status, cap = _write_side_gpu(c, keep)
    q = d["q"][0].contiguous()
    reads = {bud: _read_side_gpu(c, cache, bud, q) for bud in W.CFG4_BUDGETS}
    assert (status == 0).all() and (total == w.t_cache * keep).all()
    worst = {bud: [0.0, 0.0] for bud in W.CFG4_BUDGETS}
    for b in range(w.batch):
        x = c.cpu_sequence(b)
        kmin, kmax = O.page_meta_batch(x["k"], x["seq_len"])
        r = O.route_pack_batch(x["v"], x["scores"], None, S, keep, cap, x["seq_len"])
        o = dict(kmin=kmin, kmax=kmax, seq_len=x["seq_len"], **r)
        g1 = dict(cache=P.Cache(kmin=_slice_b(cache.kmin, b), kmax=_slice_b(cache.kmax, b),
                                v_mask=_slice_b(cache.v_mask, b), v_offs=_slice_b(cache.v_offs, b),
                                v_packed=_slice_b(cache.v_packed, b)),
                  total=_slice_b(total, b), status=_slice_b(status, b))
        H.assert_bit_exact_write_side(c.w1, g1, o)
        qb = H.cpu_bits(q[b:b + 1])
        for bud in W.CFG4_BUDGETS:
            ids, n, u = O.select_batch(qb, kmin, kmax, bud, w.t_cache, x["seq_len"], want_scores=True)
            out, lse = O.attend_batch(qb, x["k"], S, r["mask"], ids, n, H.SM_SCALE, packed=r["packed"],
                                      offs=r["offs"], seq_len=x["seq_len"])
            ob = dict(page_ids=ids, n_pages=n, u=u, out=out, lse=lse, seq_len=x["seq_len"])
            gb = {k: _slice_b(v, b) for k, v in reads[bud].items()}
            assert (n == bud // 16).all()
            H.assert_bit_exact_selection(gb, ob)
            ma, mr = H.assert_attention_close(gb, ob)
            worst[bud][0] = max(worst[bud][0], ma); worst[bud][1] = max(worst[bud][1], mr)
        del x, kmin, kmax, r, o
    print(f"cfg4 keep {keep}: worst attention error per budget {worst}")


@pytest.mark.parametrize("name,chunk", [("cfg1x32", 4), ("cfg2x28", 28)])
def test_all_layers_in_one_call(name, chunk):
    """The layer-stacked workloads (every layer's cache along the batch axis, one call per step for the
    whole model): the whole pass on the GPU at full size, every problem against the checker, `chunk`
    sequences at a time."""
    w = W.get(name)
    d = W.make_inputs(w, DEV)
    cap = w.t_cache * w.k_nominal
    g = H.gpu_pipeline(w, d, cap_groups=cap)
    assert (g["status"] == 0).all() and (g["total"] == cap).all()
    assert (g["n_pages"] == w.token_budget // 16).all()
    wc = W.shrink(w, batch=chunk)
    worst = [0.0, 0.0]
    for b0 in range(0, w.batch, chunk):
        sl = slice(b0, b0 + chunk)
        dc = dict(k=d["k"][sl], v=d["v"][sl], q=d["q"][:, sl], scores=d["scores"][sl], tok_class=None,
                  seq_len=d["seq_len"][sl])
        o = H.oracle_pipeline(wc, dc, cap_groups=cap)
        c = g["cache"]
        gc = dict(cache=P.Cache(kmin=c.kmin[sl], kmax=c.kmax[sl], v_mask=c.v_mask[sl], v_offs=c.v_offs[sl],
                                v_packed=c.v_packed[sl]),
                  total=g["total"][sl], status=g["status"][sl], page_ids=g["page_ids"][sl],
                  n_pages=g["n_pages"][sl], u=g["u"][sl], out=g["out"][sl], lse=g["lse"][sl])
        H.assert_bit_exact_write_side(wc, gc, o)
        H.assert_bit_exact_selection(gc, o)
        ma, mr = H.assert_attention_close(gc, o)
        worst = [max(worst[0], ma), max(worst[1], mr)]
        del o
    print(f"{name}: worst attention error {worst}")
