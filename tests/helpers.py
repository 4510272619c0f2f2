"""Shared plumbing for the parity tests: run the CUDA path through the C-ABI
binding, run the CPU checker on the same inputs, compare."""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle as O
import paper_2604_21335_b200 as P
from paper_2604_21335_b200 import binding as Bd

SM_SCALE = 1.0 / math.sqrt(128.0)
MAX_ABS_TOL = 1e-2          # attention outputs, bf16 inputs (stated with the metric)
MEAN_REL_TOL = 2e-3         # mean|gpu-ref| / mean|ref|


def cpu_bits(t):
    return O.bf16_bits(t.cpu())


def cpu_f32(t):
    return t.detach().float().cpu().numpy()


def gpu_pipeline(w, d, seq_len=None, budget=None, k_nominal=None, min_per_token=1, mode=Bd.MODE_GLOBAL,
                 tok_class="auto", cap_groups=None, q_index=0, want_scores=True, page_ids_override=None):
    """Full pass on the GPU: metadata, selection, routing+packing, attention.
    `d` holds CUDA tensors from workload.make_inputs.  Returns torch tensors."""
    dev = d["k"].device
    B, Hkv, T = w.batch, w.n_kv_heads, w.t_cache
    sl = d["seq_len"] if seq_len is None else torch.as_tensor(seq_len, dtype=torch.int32, device=dev)
    shape = P.Shape(B, w.n_q_heads, Hkv, w.n_groups, T, sl)
    kn = w.k_nominal if k_nominal is None else k_nominal
    cls = d["tok_class"] if isinstance(tok_class, str) else tok_class
    if cap_groups is None:
        cap_groups = T * w.n_groups
    cache = P.Cache.allocate(shape, d["k"], cap_groups)
    cache.kmin.fill_(float("nan")); cache.kmax.fill_(float("nan"))
    cache.v_packed.fill_(float("nan"))
    P.build_page_meta(shape, cache)

    total = torch.full((B, Hkv), -7, dtype=torch.int64, device=dev)
    status = torch.full((B, Hkv), -7, dtype=torch.int32, device=dev)
    ws_r = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=dev)
    ws_r.fill_(0xAB)                          # the library must not rely on a clean workspace
    P.route_pack(shape, d["v"], d["scores"], cls, kn, cache, total, status, ws_r,
                 min_per_token=min_per_token, mode=mode)

    q = d["q"][q_index].contiguous()
    bud = w.token_budget if budget is None else budget
    res = dict(shape=shape, cache=cache, total=total, status=status, q=q)
    if page_ids_override is not None:
        page_ids, n_pages = page_ids_override
    elif bud is None:
        page_ids = n_pages = None
    else:
        max_pages = max(1, min(shape.n_pages, bud // 16))
        page_ids = torch.full((B, Hkv, max_pages), -1, dtype=torch.int32, device=dev)
        n_pages = torch.full((B, Hkv), -1, dtype=torch.int32, device=dev)
        u = torch.full((B, Hkv, shape.n_pages), float("nan"), dtype=torch.float32, device=dev) if want_scores else None
        ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=dev)
        ws_s.fill_(0xCD)
        P.quest_select(shape, cache, q, bud, page_ids, n_pages, ws_s, scores=u)
        res["u"] = u
    res["page_ids"], res["n_pages"] = page_ids, n_pages
    out = torch.full((B, w.n_q_heads, 128), float("nan"), dtype=torch.float32, device=dev)
    lse = torch.full((B, w.n_q_heads), float("nan"), dtype=torch.float32, device=dev)
    mp = page_ids.shape[-1] if page_ids is not None else shape.n_pages
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, mp, device=dev)
    ws_a.fill_(0xEF)
    P.decode_attn(shape, cache, q, page_ids, n_pages, SM_SCALE, out, ws_a, lse=lse)
    torch.cuda.synchronize()
    assert int(ws_a[:4].view(torch.int32)[0]) == 0, "device status word of stc_decode_attn"
    res["out"], res["lse"] = out, lse
    return res


def oracle_pipeline(w, d, seq_len=None, budget=None, k_nominal=None, min_per_token=1, mode=O.MODE_GLOBAL,
                    tok_class="auto", cap_groups=None, q_index=0, page_ids_override=None):
    """The same pass on the CPU checker (numpy arrays in, numpy arrays out)."""
    k, v = cpu_bits(d["k"]), cpu_bits(d["v"])
    q = cpu_bits(d["q"][q_index])
    sc = d["scores"].cpu().numpy()
    T = w.t_cache
    sl = d["seq_len"].cpu().numpy() if seq_len is None else np.asarray(seq_len, np.int32)
    kn = w.k_nominal if k_nominal is None else k_nominal
    cls = d["tok_class"] if isinstance(tok_class, str) else tok_class
    cls_np = None if cls is None else cls.cpu().numpy()
    if cap_groups is None:
        cap_groups = T * w.n_groups
    kmin, kmax = O.page_meta_batch(k, sl)
    r = O.route_pack_batch(v, sc, cls_np, w.n_groups, kn, cap_groups, sl, min_per_token, mode,
                           cls_per_head=(cls_np is not None and cls_np.ndim == 3))
    bud = w.token_budget if budget is None else budget
    res = dict(kmin=kmin, kmax=kmax, seq_len=sl, **r)
    if page_ids_override is not None:
        ids, n = page_ids_override
    elif bud is None:
        ids = n = None
    else:
        ids, n, u = O.select_batch(q, kmin, kmax, bud, T, sl, want_scores=True)
        res["u"] = u
    res["page_ids"], res["n_pages"] = ids, n
    out, lse = O.attend_batch(q, k, w.n_groups, r["mask"], ids, n, SM_SCALE, packed=r["packed"],
                              offs=r["offs"], seq_len=sl)
    res["out"], res["lse"] = out, lse
    return res


def np_u16(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def assert_bit_exact_write_side(w, g, o):
    """Metadata, masks, offsets, packed store, totals: bit for bit on the valid range."""
    sl = o["seq_len"]
    S, gdim = w.n_groups, 128 // w.n_groups
    kmin_g, kmax_g = np_u16(g["cache"].kmin), np_u16(g["cache"].kmax)
    mask_g = np_u16(g["cache"].v_mask)
    offs_g = g["cache"].v_offs.cpu().numpy().view(np.uint32)
    packed_g = np_u16(g["cache"].v_packed)
    total_g, status_g = g["total"].cpu().numpy(), g["status"].cpu().numpy()
    for b in range(w.batch):
        L = int(sl[b]); Pn = (L + 15) // 16
        np.testing.assert_array_equal(kmin_g[b, :, :Pn], o["kmin"][b, :, :Pn])
        np.testing.assert_array_equal(kmax_g[b, :, :Pn], o["kmax"][b, :, :Pn])
        np.testing.assert_array_equal(mask_g[b, :, :L], o["mask"][b, :, :L])
        assert (mask_g[b, :, L:] == 0).all()
        np.testing.assert_array_equal(offs_g[b, :, :L + 1], o["offs"][b, :, :L + 1])
        np.testing.assert_array_equal(total_g[b], o["total"][b])
        for h in range(w.n_kv_heads):
            n = int(o["total"][b, h])
            assert status_g[b, h] == 0 and o["status"][b, h] == 0
            np.testing.assert_array_equal(packed_g[b, h, :n], o["packed"][b, h, :n])


def assert_bit_exact_selection(g, o, check_scores=True):
    n_g, n_o = g["n_pages"].cpu().numpy(), o["n_pages"]
    np.testing.assert_array_equal(n_g, n_o)
    ids_g = g["page_ids"].cpu().numpy()
    for b in range(n_o.shape[0]):
        for h in range(n_o.shape[1]):
            np.testing.assert_array_equal(ids_g[b, h, :n_o[b, h]], o["page_ids"][b, h, :n_o[b, h]])
    if check_scores and g.get("u") is not None:
        u_g = g["u"].cpu().numpy()
        sl = o["seq_len"]
        for b in range(n_o.shape[0]):
            Pn = (int(sl[b]) + 15) // 16
            np.testing.assert_array_equal(u_g[b, :, :Pn].view(np.uint32), o["u"][b, :, :Pn].view(np.uint32))


def attn_errors(out_gpu, out_ref):
    a = out_gpu.double().cpu().numpy() if isinstance(out_gpu, torch.Tensor) else np.asarray(out_gpu, np.float64)
    diff = np.abs(a - out_ref)
    return float(diff.max()), float(diff.mean() / max(np.abs(out_ref).mean(), 1e-30))


def assert_attention_close(g, o):
    max_abs, mean_rel = attn_errors(g["out"], o["out"])
    assert max_abs <= MAX_ABS_TOL, max_abs
    assert mean_rel <= MEAN_REL_TOL, mean_rel
    lse_g = g["lse"].double().cpu().numpy()
    fin = np.isfinite(o["lse"])
    np.testing.assert_allclose(lse_g[fin], o["lse"][fin], rtol=0, atol=2e-3)
    assert (lse_g[~fin] == o["lse"][~fin]).all()
    return max_abs, mean_rel


def near_tie_pages(u: np.ndarray, k: int, rel: float = 1e-6) -> int:
    """Pages whose bound lies within rel*max(1,|U_k|) of the k-th largest bound."""
    if k <= 0 or k >= u.shape[0]:
        return 0
    kth = np.sort(u)[::-1][k - 1]
    return int((np.abs(u - kth) <= rel * max(1.0, abs(float(kth)))).sum()) - 1
