"""stc_quest_select_static: page selection for callers that cannot allocate.

A caller that selects pages from inside a frozen memory pool, or a plugin that
only receives its input and output buffers, has no workspace to pass.  The
static variant keeps its scratch in an array inside the library, so the test
here never creates a workspace for it: it gives the call inputs and outputs only
and holds the result against what the ordinary, workspace-taking entry point
returns for the same inputs and against the CPU checker.  Calls are made back to
back with different queries, because the built-in array is shared by all calls
and still holds the previous call's counters and page scores when the next one
starts.  Two pairs of calls: one that asks for the scores (they then go to the
caller's tensor and only the counters live in the array), and one that does not,
so that the scores themselves are written to and read back from the array.

Collected last on purpose (file name), so a run that stops at the first failure
has already been through every other test.
"""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import build as B
from paper_2604_21335_b200 import workload as W


def test_shapes_beyond_the_built_in_array_are_refused_on_the_host():
    # needs no GPU: the size check comes before any device query or launch
    B.build()
    big = P.Shape(batch=64, n_q_heads=32, n_kv_heads=8, n_groups=8, t_cap=131072)
    assert P.workspace_bytes(big, Bd.OP_QUEST_SELECT) > Bd.STATIC_SCRATCH_BYTES
    lib = P.load_library()
    cs, cc = big.c(), Bd._Cache()
    rc = lib.stc_quest_select_static(cs, cc, None, 4096, 256, None, None, None, None)
    assert rc == 8
    assert b"built-in scratch" in lib.stc_status_string(rc)


@pytest.mark.gpu
def test_static_scratch_selection_matches_the_workspace_entry_point_twice_in_a_row():
    dev = "cuda"
    # Gq = 4, several CTAs per problem, ragged last page, two sequence lengths
    w = W.shrink(W.get("cfg4"), batch=2, n_q_heads=8, n_kv_heads=2, t_cache=16 * 900 + 5, token_budget=16 * 70)
    d = W.make_inputs(w, dev, n_queries=2)
    seq = torch.tensor([w.t_cache, 16 * 411 + 9], dtype=torch.int32, device=dev)
    shape = P.Shape(w.batch, w.n_q_heads, w.n_kv_heads, w.n_groups, w.t_cache, seq)
    cache = P.Cache.allocate(shape, d["k"], 1)
    P.build_page_meta(shape, cache)
    max_pages = w.token_budget // 16
    ws = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=dev)

    def fresh():
        return (torch.full((w.batch, w.n_kv_heads, max_pages), -1, dtype=torch.int32, device=dev),
                torch.full((w.batch, w.n_kv_heads), -1, dtype=torch.int32, device=dev),
                torch.full((w.batch, w.n_kv_heads, shape.n_pages), float("nan"), dtype=torch.float32, device=dev))

    kmin_c, kmax_c = O.bf16_bits(cache.kmin.cpu()), O.bf16_bits(cache.kmax.cpu())

    for call in range(2):                      # second call finds the first call's leftovers in the array
        q = d["q"][call].contiguous()
        ids_ref, n_ref, u_ref = fresh()
        P.quest_select(shape, cache, q, w.token_budget, ids_ref, n_ref, ws, scores=u_ref)
        ids, n, u = fresh()
        P.quest_select_static(shape, cache, q, w.token_budget, ids, n, scores=u)
        torch.cuda.synchronize()
        # against the CPU checker: ids, counts and score bits
        ids_o, n_o, u_o = O.select_batch(O.bf16_bits(q.cpu()), kmin_c, kmax_c, w.token_budget, w.t_cache,
                                         seq.cpu().numpy(), want_scores=True)
        np.testing.assert_array_equal(n.cpu().numpy(), n_o)
        np.testing.assert_array_equal(ids.cpu().numpy(), ids_o)
        for b in range(w.batch):
            npg = (int(seq[b]) + 15) // 16
            np.testing.assert_array_equal(u[b, :, :npg].cpu().numpy().view(np.uint32),
                                          u_o[b, :, :npg].view(np.uint32))
        # integer outputs and the fp32 scores that decide them: bit for bit
        assert torch.equal(n, n_ref) and int(n_ref.min()) == max_pages
        assert torch.equal(ids, ids_ref)
        valid = torch.arange(shape.n_pages, device=dev)[None, None, :] < ((seq + 15) // 16)[:, None, None]
        assert torch.equal(u.view(torch.int32)[valid.expand_as(u)], u_ref.view(torch.int32)[valid.expand_as(u)])
        if call == 1:
            assert not torch.equal(ids, first_ids)     # the two queries really select different pages
        first_ids = ids


@pytest.mark.gpu
def test_static_scratch_holds_the_scores_when_the_caller_passes_none():
    """Without a score tensor the fp32 page scores live in the built-in array: the second call
    starts with the first query's scores still there and must not be influenced by them."""
    dev = "cuda"
    # several CTAs per problem, ragged lengths: Gq = 4 with 4300 pages (the tensor-core scan, whose approximate
    # scores and per-problem words live in the array) and Gq = 1 with 1800 pages (the fp32 scan)
    for hq, hkv, pages in ((8, 2, 4300), (3, 3, 1800)):
        w = W.shrink(W.get("cfg4"), batch=2, n_q_heads=hq, n_kv_heads=hkv, t_cache=16 * pages + 11,
                     token_budget=16 * 130)
        d = W.make_inputs(w, dev, n_queries=3)
        seq = torch.tensor([w.t_cache, 16 * 977 + 2], dtype=torch.int32, device=dev)
        shape = P.Shape(w.batch, w.n_q_heads, w.n_kv_heads, w.n_groups, w.t_cache, seq)
        cache = P.Cache.allocate(shape, d["k"], 1)
        P.build_page_meta(shape, cache)
        max_pages = w.token_budget // 16
        ws = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=dev)
        kmin_c, kmax_c = O.bf16_bits(cache.kmin.cpu()), O.bf16_bits(cache.kmax.cpu())
        prev = None
        for call in range(3):
            q = d["q"][call].contiguous()
            ids_ref = torch.full((w.batch, w.n_kv_heads, max_pages), -1, dtype=torch.int32, device=dev)
            n_ref = torch.full((w.batch, w.n_kv_heads), -1, dtype=torch.int32, device=dev)
            ids, n = torch.full_like(ids_ref, -1), torch.full_like(n_ref, -1)
            P.quest_select(shape, cache, q, w.token_budget, ids_ref, n_ref, ws)
            P.quest_select_static(shape, cache, q, w.token_budget, ids, n)
            torch.cuda.synchronize()
            assert torch.equal(n, n_ref) and torch.equal(ids, ids_ref)
            ids_o, n_o = O.select_batch(O.bf16_bits(q.cpu()), kmin_c, kmax_c, w.token_budget, w.t_cache,
                                        seq.cpu().numpy())
            np.testing.assert_array_equal(n.cpu().numpy(), n_o)
            np.testing.assert_array_equal(ids.cpu().numpy(), ids_o)
            if prev is not None:
                assert not torch.equal(ids, prev)
            prev = ids
