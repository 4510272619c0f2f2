"""A decode loop under a running group budget: tokens are appended at full width
(stc_append_tokens) and every page that completes is routed on its own (stc_route_new_pages), so the
routed tokens always hold exactly N*K groups (Section 3.4, Appendix B.1) while the open page stays
uncompressed.  The cache the loop ends in must equal, bit for bit, the one the CPU checker builds
WITHOUT any in-place step (the prefix routed as a whole, each later page routed alone, the tail at
full width, packed in one sequential walk), and selection + attention on it must match."""
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

CASES = [
    # name, overrides, prefix lengths, steps, route every, mode, floor
    ("cfg2", dict(batch=2, t_cache=16 * 40, token_budget=16 * 12), [16 * 20 + 3, 16 * 11 + 15], 70, 1, 0, 1),   # S16 K4 Gq7
    ("cfg0", dict(n_q_heads=2, n_kv_heads=2, batch=3, t_cache=16 * 40 + 5, token_budget=16 * 9),
     [16 * 9, 16 * 3 + 8, 1], 100, 37, 0, 1),                                                             # pages pile up
    ("cfg0", dict(n_q_heads=4, n_kv_heads=2, batch=2, t_cache=16 * 30, token_budget=16 * 8, n_groups=4, k_nominal=1),
     [16 * 5 + 1, 16 * 7 + 9], 60, 1, 1, 1),                                                              # S4K1 per token
    ("cfg0", dict(n_q_heads=2, n_kv_heads=2, batch=2, t_cache=16 * 30, token_budget=16 * 8, k_nominal=2),
     [16 * 4 + 7, 16 * 6], 50, 16, 0, 0),                                                                 # no floor
]


@pytest.mark.parametrize("name,over,prefix,steps,every,mode,mpt", CASES)
def test_decode_loop_keeps_the_running_budget(name, over, prefix, steps, every, mode, mpt):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV, n_queries=2)
    B, Hkv, T, S, K = w.batch, w.n_kv_heads, w.t_cache, w.n_groups, w.k_nominal
    d["scores"] = torch.round(d["scores"] * 4) / 4                    # ties inside pages
    cur = torch.tensor(prefix, dtype=torch.int32, device=DEV)
    shape = P.Shape(B, w.n_q_heads, Hkv, S, T, cur)
    cache = P.Cache.allocate(shape, d["k"], T * S)
    cache.v_packed.fill_(float("nan"))
    total = torch.zeros(B, Hkv, dtype=torch.int64, device=DEV)
    status = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    # prefix: complete pages routed as a whole, the open page at full width
    cls0 = torch.zeros(B, T, dtype=torch.uint8, device=DEV)
    for b, L in enumerate(prefix):
        cls0[b, :(L // 16) * 16] = Bd.CLS_ROUTED
        cls0[b, (L // 16) * 16:L] = Bd.CLS_FULL
    P.build_page_meta(shape, cache)
    P.route_pack(shape, d["v"], d["scores"], cls0, K, cache, total, status,
                 Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV), min_per_token=mpt, mode=mode)
    first = torch.tensor([L // 16 for L in prefix], dtype=torch.int32, device=DEV)
    lens = list(prefix)
    for step in range(1, steps + 1):
        old_len = cur.clone()
        cur += 1
        lens = [x + 1 for x in lens]
        P.append_tokens(shape, cache, d["v"], old_len, 1, total, status)
        if step % every == 0 or step == steps:
            P.route_new_pages(shape, cache, d["scores"], first, K, total, status, min_per_token=mpt, mode=mode)
            first = torch.tensor([L // 16 for L in lens], dtype=torch.int32, device=DEV)
            torch.cuda.synchronize()
            assert (status == 0).all(), status
            want_total = torch.tensor([[(L // 16) * 16 * K + (L % 16) * S] * Hkv for L in lens], device=DEV)
            assert torch.equal(total, want_total)                   # N*K over the routed tokens + the open page
    # the checker's construction of the final state
    sl = np.asarray(lens, np.int32)
    sc = d["scores"].cpu().numpy()
    k_bits, v_bits = H.cpu_bits(d["k"]), H.cpu_bits(d["v"])
    r0 = O.route_pack_batch(v_bits, sc, cls0.cpu().numpy(), S, K, T * S, np.asarray(prefix, np.int32), mpt, mode)
    mask = np.zeros((B, Hkv, T), np.uint16)
    offs = np.zeros((B, Hkv, T + 1), np.uint32)
    packed = np.zeros((B, Hkv, T * S, 128 // S), np.uint16)
    tot = np.zeros((B, Hkv), np.int64)
    for b in range(B):
        p0, L = prefix[b] // 16, lens[b]
        for h in range(Hkv):
            m = mask[b, h]
            m[:p0 * 16] = r0["mask"][b, h, :p0 * 16]
            for p in range(p0, L // 16):
                rc, mp_ = O.route(sc[b, h, 16 * p:16 * p + 16], None, S, K, mpt, mode)
                assert rc == 0
                m[16 * p:16 * p + 16] = mp_
            m[(L // 16) * 16:L] = (1 << S) - 1
            n, of, pk = O.pack(v_bits[b, h, :L], m[:L], S, T * S)
            offs[b, h, :L + 1] = of; packed[b, h] = pk; tot[b, h] = n
    kmin, kmax = O.page_meta_batch(k_bits, sl)
    o = dict(kmin=kmin, kmax=kmax, seq_len=sl, mask=mask, offs=offs, packed=packed, total=tot,
             status=np.zeros((B, Hkv), np.int32))
    H.assert_bit_exact_write_side(w, dict(cache=cache, total=total, status=status), o)

    # read side on the cache the loop produced
    q = d["q"][1].contiguous()
    mp = w.token_budget // 16
    ids = torch.full((B, Hkv, mp), -1, dtype=torch.int32, device=DEV)
    npg = torch.full((B, Hkv), -1, dtype=torch.int32, device=DEV)
    P.quest_select(shape, cache, q, w.token_budget, ids, npg, Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=DEV))
    out = torch.zeros(B, w.n_q_heads, 128, dtype=torch.float32, device=DEV)
    lse = torch.zeros(B, w.n_q_heads, dtype=torch.float32, device=DEV)
    P.decode_attn(shape, cache, q, ids, npg, H.SM_SCALE, out,
                  Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, mp, device=DEV), lse=lse)
    torch.cuda.synchronize()
    qb = H.cpu_bits(q)
    ids_o, n_o = O.select_batch(qb, kmin, kmax, w.token_budget, T, sl)
    out_o, lse_o = O.attend_batch(qb, k_bits, S, mask, ids_o, n_o, H.SM_SCALE, packed=packed, offs=offs, seq_len=sl)
    H.assert_bit_exact_selection(dict(page_ids=ids, n_pages=npg), dict(page_ids=ids_o, n_pages=n_o, seq_len=sl),
                                 check_scores=False)
    H.assert_attention_close(dict(out=out, lse=lse), dict(out=out_o, lse=lse_o))


def test_refusals_leave_the_cache_alone():
    w = W.shrink(W.get("cfg0"), n_q_heads=2, n_kv_heads=2, batch=2, t_cache=16 * 30)
    d = W.make_inputs(w, DEV)
    cur = torch.tensor([16 * 12, 16 * 20 + 3], dtype=torch.int32, device=DEV)
    shape = P.Shape(2, 2, 2, w.n_groups, w.t_cache, cur)
    cache = P.Cache.allocate(shape, d["k"], w.t_cache * 8)
    total = torch.zeros(2, 2, dtype=torch.int64, device=DEV)
    status = torch.zeros(2, 2, dtype=torch.int32, device=DEV)
    cls = torch.full((2, w.t_cache), Bd.CLS_FULL, dtype=torch.uint8, device=DEV)
    cls[1, :16 * 18] = Bd.CLS_ROUTED
    P.route_pack(shape, d["v"], d["scores"], cls, 4, cache, total, status,
                 Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV))
    before = (cache.v_mask.clone(), cache.v_offs.clone(), cache.v_packed.clone(), total.clone())
    # sequence 0: 12 completed pages at once (more than a call takes); sequence 1: page 17 is already routed
    first = torch.tensor([0, 17], dtype=torch.int32, device=DEV)
    P.route_new_pages(shape, cache, d["scores"], first, 4, total, status)
    torch.cuda.synchronize()
    assert (status == 1).all()
    # floor of one group per token with a budget of zero groups
    first = torch.tensor([6, 18], dtype=torch.int32, device=DEV)
    P.route_new_pages(shape, cache, d["scores"], first, 0, total, status)
    torch.cuda.synchronize()
    assert (status == 5).all()
    for a, b in zip(before, (cache.v_mask, cache.v_offs, cache.v_packed, total)):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                           b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
