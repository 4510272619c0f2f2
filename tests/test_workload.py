"""The seeded input generator: counter-based, so the CPU and the GPU draw the same bits and any
subset of problems can be drawn alone.  (It holds none of the method's arithmetic.)"""
import pytest
import torch

from paper_2604_21335_b200 import workload as W


def _fmix(x):
    x &= 0xFFFFFFFF; x ^= x >> 16; x = (x * 0x85EBCA6B) & 0xFFFFFFFF
    x ^= x >> 13; x = (x * 0xC2B2AE35) & 0xFFFFFFFF
    return x ^ (x >> 16)


def test_elements_follow_the_integer_hash_and_the_normal_table():
    w = W.shrink(W.get("cfg0"), t_cache=300)
    d = W.make_inputs(w, "cpu")
    tab = W._normal_table()
    assert abs(float(tab.double().mean())) < 1e-6 and abs(float(tab.double().std()) - 1.0) < 1e-3
    for tensor_id, name, hk in [(W._T_V, "v", 5), (W._T_V, "v", 0)]:
        ka, kb = W._keys(w.seed, tensor_id, hk)
        flat = d[name][0, hk].flatten()
        for i in (0, 1, 77, 300 * 128 - 1):
            h = _fmix((_fmix((i ^ ka) & 0xFFFFFFFF) + kb) & 0xFFFFFFFF)
            assert flat[i] == tab[h >> 16].to(torch.bfloat16)
    # four outlier channels per head, scaled by 8
    std = d["k"][0, 2].float().std(0)
    assert int((std > 4).sum()) == 4


def test_a_subset_of_problems_equals_the_slices_of_the_full_draw():
    w = W.shrink(W.get("cfg2"), batch=3, t_cache=200)
    d = W.make_inputs(w, "cpu", n_queries=2)
    ps = [(0, 3), (2, 1)]
    s = W.make_inputs(w, "cpu", n_queries=2, problems=ps)
    w1 = W.problem_view(w, ps)
    assert (w1.batch, w1.n_kv_heads, w1.n_q_heads) == (2, 1, 7)
    for i, (b, h) in enumerate(ps):
        assert torch.equal(s["k"][i, 0].view(torch.int16), d["k"][b, h].view(torch.int16))
        assert torch.equal(s["v"][i, 0].view(torch.int16), d["v"][b, h].view(torch.int16))
        assert torch.equal(s["scores"][i, 0], d["scores"][b, h])
        assert torch.equal(s["q"][:, i].view(torch.int16), d["q"][:, b, 7 * h:7 * h + 7].view(torch.int16))


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["cfg1", "cfg3"])
def test_cpu_and_gpu_draw_the_same_bits(name):
    w = W.shrink(W.get(name), batch=2, n_q_heads=4, n_kv_heads=4, t_cache=272)
    a, b = W.make_inputs(w, "cpu", n_queries=2), W.make_inputs(w, "cuda", n_queries=2)
    for key in ("k", "v", "q"):
        assert torch.equal(a[key].view(torch.int16), b[key].cpu().view(torch.int16)), key
    assert torch.equal(a["scores"].view(torch.int32), b["scores"].cpu().view(torch.int32))
    assert (a["tok_class"] is None) == (b["tok_class"] is None)
    if a["tok_class"] is not None:
        assert torch.equal(a["tok_class"], b["tok_class"].cpu())
