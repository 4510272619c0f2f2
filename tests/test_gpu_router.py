"""Router logits (tcgen05 GEMM) against the CPU checker: fp32 accumulation of exact bf16
products, so the tolerance is a few ulps of the accumulated magnitude."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2604_21335_b200 as P

import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_case(B, T, Hkv, S, dm, with_bias, seed):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    h = torch.randn(B, T, dm, generator=g, device=DEV).to(torch.bfloat16)
    w = (torch.randn(Hkv * S, dm, generator=g, device=DEV) / dm ** 0.5).to(torch.bfloat16)
    bias = torch.randn(B, Hkv * S, generator=g, device=DEV) if with_bias else None
    shape = P.Shape(B, Hkv, Hkv, S, T)
    scores = torch.full((B, Hkv, T, S), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    P.router_logits(shape, h, w, scores, status, bias=bias)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    want = O.router_logits(H.cpu_bits(h), H.cpu_bits(w), S, None if bias is None else bias.cpu().numpy())
    got = scores.double().cpu().numpy()
    # |error| <= K * 2^-24 * sum|h||w| is the worst case of an fp32 sum; allow a tenth of that bound
    bound = float((h.float().abs() @ w.float().abs().T).max()) * dm * 2.0 ** -24
    err = np.abs(got - want).max()
    assert np.isfinite(got).all() and err <= max(0.1 * bound, 1e-5), (err, bound)
    return err


@pytest.mark.parametrize("B,T,Hkv,S,dm,bias", [
    (1, 128, 8, 8, 64, False),          # one tile, one K slice
    (1, 256, 8, 8, 256, False),         # two tiles, four K slices (ring not yet wrapped)
    (2, 300, 4, 16, 1024, True),        # ragged last tile, ring wraps, bias, S = 16
    (1, 1000, 32, 8, 4096, True),       # LLaMA-2-7B router: 256 logits, d_model 4096
    (3, 77, 4, 4, 512, False),          # 16 logits, S = 4, tokens of several sequences in one tile
    (1, 200, 64, 8, 128, True),         # 512 logits: two column tiles
])
def test_router_logits_match_the_checker(B, T, Hkv, S, dm, bias):
    run_case(B, T, Hkv, S, dm, bias, seed=B * 1000 + T)


def test_unsupported_shapes_are_refused_on_the_host():
    shape = P.Shape(1, 1, 1, 8, 64)                       # 8 logits: not a multiple of 16
    x = torch.zeros(1, 64, 64, dtype=torch.bfloat16, device=DEV)
    w = torch.zeros(8, 64, dtype=torch.bfloat16, device=DEV)
    sc = torch.zeros(1, 1, 64, 8, device=DEV); st = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(P.StcError) as e:
        P.router_logits(shape, x, w, sc, st)
    assert e.value.code == 2


@pytest.mark.parametrize("B,Lq,dm,N", [
    (1, 1, 64, 16),                     # one token: the mean is the row
    (3, 37, 4096, 256),                 # LLaMA-2-7B router width, ragged region lengths
    (2, 130, 264, 64),                  # d_model not a multiple of the 256-channel CTA slice
])
def test_query_summary_term_matches_the_checker_and_feeds_the_router(B, Lq, dm, N):
    g = torch.Generator(device=DEV); g.manual_seed(B * 100 + Lq)
    h_q = torch.randn(B, Lq, dm, generator=g, device=DEV).to(torch.bfloat16)
    w_q = (torch.randn(N, dm, generator=g, device=DEV) / dm ** 0.5).to(torch.bfloat16)
    q_len = torch.tensor([Lq, max(Lq // 3, 0), 0][:B], dtype=torch.int32, device=DEV)
    s_q = torch.full((B, dm), float("nan"), dtype=torch.float32, device=DEV)
    bias = torch.full((B, N), float("nan"), dtype=torch.float32, device=DEV)
    P.query_bias(h_q, w_q, s_q, bias, q_len=q_len)
    torch.cuda.synchronize()
    s_o, b_o = O.query_bias(H.cpu_bits(h_q), H.cpu_bits(w_q), q_len.cpu().numpy())
    # fp32 sums of n terms: worst case n * 2^-24 * sum|terms|; allow a tenth of it
    mean_abs = np.stack([np.abs(H.cpu_f32(h_q)[b, : int(q_len[b])]).mean(axis=0) if int(q_len[b]) else np.zeros(dm)
                         for b in range(B)])
    tol_s = 0.1 * Lq * 2.0 ** -24 * mean_abs.max() + 1e-7
    assert np.abs(s_q.double().cpu().numpy() - s_o).max() <= tol_s
    tol_b = 0.1 * (dm + Lq) * 2.0 ** -24 * float((mean_abs @ np.abs(H.cpu_f32(w_q)).T).max()) + 1e-7
    assert np.abs(bias.double().cpu().numpy() - b_o).max() <= tol_b
    # a second call gives the same bits (fixed summation order)
    s2, b2 = torch.empty_like(s_q), torch.empty_like(bias)
    P.query_bias(h_q, w_q, s2, b2, q_len=q_len)
    assert torch.equal(s2, s_q) and torch.equal(b2, bias)
