"""Seeded random shapes through the whole path: group counts, head groupings, lengths from one
token to a dozen thousand (both selection kernels, CTA ranges inside and across problems),
ragged and empty sequences, class mixes, both routing modes, budgets from zero to all groups,
continuous and heavily tied scores.  Every case against the CPU checker: integer outputs bit
for bit, attention within the stated tolerance.  Each seed runs twice: with the routing selection
kernel the library would pick for the size (the multi-pass kernel at these sizes) and with the band
kernel forced through the library's test-only launch parameter."""
import ctypes as C
import random

import numpy as np
import pytest
import torch

import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import workload as W

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def knobs(first_pass):
    lib = P.load_library()
    lib.stc_test_route_select_knobs.restype = None
    lib.stc_test_route_select_knobs.argtypes = [C.c_int32, C.c_uint64]
    lib.stc_test_route_select_knobs(first_pass, 0)


@pytest.mark.parametrize("knob", [0, 7])
@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_cases_match_the_checker(seed, knob):
    knobs(knob)
    try:
        run_cases(seed)
    finally:
        knobs(0)


def run_cases(seed):
    rnd = random.Random(seed)
    compared = 0
    for case in range(16):
        S = rnd.choice([4, 8, 16]); Hkv = rnd.choice([1, 2, 4]); gq = rnd.choice([1, 2, 4, 7]); B = rnd.choice([1, 2, 5, 9])
        T = rnd.choice([rnd.randint(1, 300), rnd.randint(300, 3000), rnd.randint(3000, 12000)])
        kn = rnd.randint(0, S); mpt = rnd.choice([0, 1]); mode = rnd.choice([0, 0, 0, 1])
        if mode == 1:
            kn = max(kn, 1)
        recipe = rnd.choice(["normal", "vnorm", "ties"])
        w = W.Workload("fuzz", B, Hkv * gq, Hkv, T, S, kn, 16 * rnd.randint(1, 40),
                       "normal" if recipe == "ties" else recipe, seed=rnd.randint(0, 1 << 30))
        d = W.make_inputs(w, DEV)
        if recipe == "ties":
            g0 = torch.Generator(device="cpu"); g0.manual_seed(seed * 1000 + case)
            d["scores"] = (torch.randint(-2, 3, d["scores"].shape, generator=g0).float()
                           * rnd.choice([1.0, 0.0, 0.5])).to(DEV)
        seq = torch.tensor([rnd.choice([T, rnd.randint(0, T), 0 if rnd.random() < 0.1 else rnd.randint(1, T)])
                            for _ in range(B)], dtype=torch.int32)
        cls = None
        if rnd.random() < 0.5:
            cls = torch.tensor(np.random.RandomState(seed * 1000 + case).randint(0, 3, (B, T)), dtype=torch.uint8)
        g = H.gpu_pipeline(w, d, seq_len=seq.to(DEV), tok_class=None if cls is None else cls.to(DEV), k_nominal=kn,
                           min_per_token=mpt, mode=mode)
        o = H.oracle_pipeline(w, d, seq_len=seq.numpy(), tok_class=cls, k_nominal=kn, min_per_token=mpt, mode=mode)
        if (o["status"] == 0).all():
            H.assert_bit_exact_write_side(w, g, o)
            H.assert_bit_exact_selection(g, o)
            H.assert_attention_close(g, o)
            compared += 1
        else:                                            # budget below one group per token somewhere: both sides say so
            assert ((g["status"].cpu().numpy() != 0) == (o["status"] != 0)).all()
    assert compared >= 10
