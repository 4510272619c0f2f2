"""The give-up path of the one kernel in which CTAs wait for each other (the cooperative selection
kernel of stc_route_pack): its hand-off waits are bounded, and a wait that runs out must end the
kernel in an orderly way, report STC_ERR_TIMEOUT for every problem and leave the library usable.

Nothing here hangs or faults the GPU: a test-only launch parameter starts the kernel at its mask pass
on a freshly cleared workspace, where no CTA will ever publish a threshold, and bounds every wait by
one millisecond, so each CTA's wait simply expires and the CTA returns."""
import ctypes as C

import pytest
import torch

import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd
from paper_2604_21335_b200 import workload as W

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def knobs(first_pass, wait_ns):
    lib = P.load_library()
    lib.stc_test_route_select_knobs.restype = None
    lib.stc_test_route_select_knobs.argtypes = [C.c_int32, C.c_uint64]
    lib.stc_test_route_select_knobs(first_pass, wait_ns)


@pytest.mark.parametrize("name,over", [("cfg1", dict(n_q_heads=4, n_kv_heads=4, t_cache=6000)),
                                       ("cfg2", dict(batch=3, t_cache=4100))])
def test_expired_hand_off_wait_reports_timeout_and_the_next_call_is_exact(name, over):
    w = W.shrink(W.get(name), **over)
    d = W.make_inputs(w, DEV)
    ref = H.gpu_pipeline(w, d)                               # an ordinary pass: the expected result
    o = H.oracle_pipeline(w, d)
    H.assert_bit_exact_write_side(w, ref, o)
    shape = ref["shape"]
    cap = ref["cache"].cap_groups
    cache = P.Cache.allocate(shape, d["k"], cap)
    total = torch.full_like(ref["total"], -7)
    status = torch.full_like(ref["status"], -7)
    ws = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=DEV)
    ws.fill_(0x3C)
    try:
        knobs(3, 1_000_000)                                  # start at the mask pass, waits give up after 1 ms
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        P.route_pack(shape, d["v"], d["scores"], d["tok_class"], w.k_nominal, cache, total, status, ws)
        t1.record()
        torch.cuda.synchronize()
    finally:
        knobs(0, 0)                                          # back to the defaults
    assert (status == 7).all(), status                       # STC_ERR_TIMEOUT in every entry
    assert t0.elapsed_time(t1) < 500.0                       # the waits ended at their limit, nothing spun on
    # the same workspace and buffers, an ordinary call right after: bit for bit the expected result
    P.route_pack(shape, d["v"], d["scores"], d["tok_class"], w.k_nominal, cache, total, status, ws)
    torch.cuda.synchronize()
    g = dict(cache=cache, total=total, status=status)
    cache.kmin, cache.kmax = ref["cache"].kmin, ref["cache"].kmax
    H.assert_bit_exact_write_side(w, g, o)
