"""Every way stc_route_pack settles the global budget gives the checker's masks, bit for bit.

The library has two kernels for it: the band kernel (a sampled histogram proposes a band of scores
around the threshold, one full scan lists the pairs inside it and counts the pairs above, the exact
count check accepts or rejects the band) and the multi-pass radix kernel, which also takes over the
problems whose band was rejected or whose list overflowed.  A test-only launch parameter (not in the
public header) selects among them; the result must not depend on it.
   0  production: the band kernel for score arrays of half the L2 size and beyond (then the multi-pass kernel
      for what it left), the multi-pass kernel alone for smaller ones
   7  the production band kernel whatever the size
  -1  multi-pass kernel alone
   5  band kernel with every token in the sample (the band is exact)
   6  band kernel with a band of almost no width: most bands miss, those problems are redone
"""
import ctypes as C

import pytest
import torch

import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import workload as W

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def knobs(first_pass, wait_ns=0):
    lib = P.load_library()
    lib.stc_test_route_select_knobs.restype = None
    lib.stc_test_route_select_knobs.argtypes = [C.c_int32, C.c_uint64]
    lib.stc_test_route_select_knobs(first_pass, wait_ns)


# problems long enough for the sample to be a real one (T * S >= 2^18 keys), few of them so the checker is quick
CASES = [
    ("cfg1", dict(n_q_heads=2, n_kv_heads=2, t_cache=40000, token_budget=512), None, {}),                 # one token in 2
    ("cfg2", dict(batch=2, n_q_heads=14, n_kv_heads=2, t_cache=33000, token_budget=512), [33000, 20011], {}),  # one in 4, ragged
    ("cfg4", dict(batch=1, n_q_heads=8, n_kv_heads=2, t_cache=131072, token_budget=512), None, {}),       # one in 8
    ("cfg4", dict(batch=1, n_q_heads=4, n_kv_heads=1, t_cache=131072 + 300, token_budget=512, k_nominal=2), None,
     dict(min_per_token=0)),
    ("cfg1", dict(n_q_heads=2, n_kv_heads=2, t_cache=9000, token_budget=512), None, {}),                  # every token (short)
]


@pytest.mark.parametrize("knob", [0, 7, -1, 5, 6])
@pytest.mark.parametrize("name,over,seq,kw", CASES)
def test_masks_do_not_depend_on_the_selection_kernel(name, over, seq, kw, knob):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV)
    o = H.oracle_pipeline(w, d, seq_len=seq, **kw)
    try:
        knobs(knob)
        g = H.gpu_pipeline(w, d, seq_len=seq, **kw)
        torch.cuda.synchronize()
    finally:
        knobs(0)
    H.assert_bit_exact_write_side(w, g, o)


@pytest.mark.parametrize("knob", [7, 5, 6])
def test_massive_ties_and_skewed_scores(knob):
    w = W.shrink(W.get("cfg1"), n_q_heads=3, n_kv_heads=3, t_cache=40000, token_budget=512)
    d = W.make_inputs(w, DEV)
    s = d["scores"]
    s[0, 0] = torch.round(s[0, 0] * 2) / 2                  # a handful of distinct values: the list overflows
    s[0, 1] = 0.25                                          # every pair ties
    s[0, 2, :20000] += 3.0                                  # the first half scores higher: a block sample would be off
    s[0, 2, 100:200] = -0.0
    o = H.oracle_pipeline(w, d)
    try:
        knobs(knob)
        g = H.gpu_pipeline(w, d)
        torch.cuda.synchronize()
    finally:
        knobs(0)
    H.assert_bit_exact_write_side(w, g, o)


@pytest.mark.parametrize("step", [4096.0, 256.0, 32.0])
def test_ties_on_the_threshold_inside_the_band(step):
    """Scores on a grid: with 4096 steps per unit a few dozen pairs share the threshold value, with 256 several
    hundred (both ranked by flat index in the settle kernel), with 32 several thousand (too many to rank there:
    the multi-pass kernel redoes the problem)."""
    w = W.shrink(W.get("cfg1"), n_q_heads=2, n_kv_heads=2, t_cache=40000, token_budget=512)
    d = W.make_inputs(w, DEV)
    d["scores"] = torch.round(d["scores"] * step) / step
    o = H.oracle_pipeline(w, d)
    try:
        knobs(7)
        g = H.gpu_pipeline(w, d)
        torch.cuda.synchronize()
    finally:
        knobs(0)
    H.assert_bit_exact_write_side(w, g, o)


@pytest.mark.parametrize("knob", [7, 5, -1])
def test_signed_zeros_and_infinities_around_the_threshold(knob):
    """The scores are shifted so that the budget's threshold is zero, then sprinkled with +0, -0 (equal as keys),
    +inf and -inf: the band's edges sit next to zero, the pairs on the threshold carry both signs of zero."""
    w = W.shrink(W.get("cfg1"), n_q_heads=2, n_kv_heads=2, t_cache=40000, token_budget=512)
    d = W.make_inputs(w, DEV)
    s = d["scores"]
    T, S, K = w.t_cache, w.n_groups, w.k_nominal
    gen = torch.Generator(device="cpu").manual_seed(5)
    for h in range(2):
        rest = torch.sort(s[0, h], dim=1, descending=True).values[:, 1:].reshape(-1)   # all but each token's maximum
        kth = torch.topk(rest, T * (K - 1)).values[-1]
        s[0, h] -= kth                                       # the (N K - N)-th largest remaining score is now +0
        flat = s[0, h].view(-1)
        idx = torch.randperm(T * S, generator=gen)[:1200].to(flat.device)
        flat[idx[:300]] = 0.0
        flat[idx[300:600]] = -0.0
        flat[idx[600:900]] = float("inf")
        flat[idx[900:]] = float("-inf")
    o = H.oracle_pipeline(w, d)
    try:
        knobs(knob)
        g = H.gpu_pipeline(w, d)
        torch.cuda.synchronize()
    finally:
        knobs(0)
    H.assert_bit_exact_write_side(w, g, o)


def test_band_kernel_wait_expires_in_an_orderly_way():
    """Without its first scan nobody publishes a band, so every wait of the band kernel runs into its limit."""
    w = W.shrink(W.get("cfg1"), n_q_heads=4, n_kv_heads=4, t_cache=6000)
    d = W.make_inputs(w, DEV)
    ref = H.gpu_pipeline(w, d)
    o = H.oracle_pipeline(w, d)
    H.assert_bit_exact_write_side(w, ref, o)
    shape = ref["shape"]
    cache = P.Cache.allocate(shape, d["k"], ref["cache"].cap_groups)
    total = torch.full_like(ref["total"], -7)
    status = torch.full_like(ref["status"], -7)
    ws = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV)
    ws.fill_(0x3C)
    try:
        knobs(4, 1_000_000)
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        P.route_pack(shape, d["v"], d["scores"], d["tok_class"], w.k_nominal, cache, total, status, ws)
        t1.record()
        torch.cuda.synchronize()
    finally:
        knobs(0, 0)
    assert (status == 7).all(), status                       # STC_ERR_TIMEOUT in every entry
    assert t0.elapsed_time(t1) < 500.0
    P.route_pack(shape, d["v"], d["scores"], d["tok_class"], w.k_nominal, cache, total, status, ws)
    torch.cuda.synchronize()
    g = dict(cache=cache, total=total, status=status)
    cache.kmin, cache.kmax = ref["cache"].kmin, ref["cache"].kmax
    H.assert_bit_exact_write_side(w, g, o)
