#!/usr/bin/env python
"""Benchmark of the sub-token-routed decode path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input:
  stc_build_page_meta -> stc_route_pack -> stc_quest_select -> stc_decode_attn
(the write side and the read side, each once).  The metric is decode-attention
GB/s: ALGORITHMIC bytes (what the method itself must move: keys read for the
metadata, router scores once, kept value groups in and out, page metadata,
selected keys, packed values, masks, offsets and page ids) divided by device
time.  Every call is bracketed by CUDA events on the launching stream inside
the timed region, so the line also carries per-call GB/s and the roofline
fraction of the dominant kernel against the measured copy bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1]
  python bench.py --impl reference ...       # the CPU checker, timed as it stands
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2604_21335_b200 import dist as D  # noqa: E402
from paper_2604_21335_b200 import workload as W  # noqa: E402

METRIC = "decode_attention_GBps"
UNIT = "GB/s"
SM_SCALE = 1.0 / math.sqrt(128.0)
FALLBACK_HBM_GBS = 6650.0        # earlier measurement on this machine, used only without MEASURED_PEAKS.json
NOMINAL_HBM_GBS = 8000.0


# --------------------------------------------------------------------------- bytes
def algorithmic_bytes(w: W.Workload, seq_len, n_routed, n_full, total_groups, sel_pages, sel_tokens,
                      sel_groups) -> dict:
    """Per-call algorithmic bytes of one step (ints, summed over all problems)."""
    g2 = w.group_dim * 2
    Hkv, Hq = w.n_kv_heads, w.n_q_heads
    tok = int(sum(seq_len)) * Hkv                               # (problem, token) rows
    pages = int(sum((n + 15) // 16 for n in seq_len)) * Hkv
    meta = tok * 256 + pages * 512
    route = (n_routed * w.n_groups * 4                         # router scores, once
             + (tok if w.n_text else 0)                         # token classes
             + tok * 2)                                         # masks
    pack = total_groups * g2 * 2 + (tok + w.n_problems) * 4    # kept groups in + out, offsets
    q_out = w.batch * Hq * (256 + 512)
    select = 0
    if w.token_budget is not None:
        select = pages * 512 + w.batch * Hq * 256 + sel_pages * 4 + w.n_problems * 4
    attn = sel_tokens * 256 + sel_groups * g2 + sel_tokens * 2 + sel_pages * 8 + q_out
    return dict(page_meta=meta, route_mask=route, pack_values=pack, quest_select=select, decode_attn=attn)


def peaks() -> tuple[float, str]:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# -------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _once(self):
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            try:
                bits = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            except Exception:
                bits = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            for b, name in self.REASONS.items():
                if bits & b:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._once()
            self._stop.wait(self.period)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self) -> dict:
        if self._thr:
            self._once()
            self._stop.set()
            self._thr.join()
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------- CPU checker
def oracle_step(w: W.Workload, d_cpu: dict, problems: list, q_index: int = 0) -> dict:
    """One pass of the CPU checker over the listed (batch, kv head) problems.
    Returns wall seconds and the same algorithmic byte count as the GPU arm."""
    import numpy as np
    import oracle as O
    gq = w.gq
    bs = sorted({b for b, _ in problems})
    work = []
    for b in bs:                           # slice the sample out before the clock starts
        hs = [h for bb, h in problems if bb == b]
        work.append(dict(
            k=np.ascontiguousarray(d_cpu["k"][b:b + 1, hs]), v=np.ascontiguousarray(d_cpu["v"][b:b + 1, hs]),
            sc=np.ascontiguousarray(d_cpu["scores"][b:b + 1, hs]),
            q=np.ascontiguousarray(np.concatenate(
                [d_cpu["q"][q_index, b:b + 1, h * gq:(h + 1) * gq] for h in hs], axis=1)),
            cls=None if d_cpu["tok_class"] is None else d_cpu["tok_class"][b:b + 1],
            sl=d_cpu["seq_len"][b:b + 1]))
    t0 = time.perf_counter()
    # one batch element at a time, so the batched drivers (OpenMP over problems) are used
    for x in work:
        kmin, kmax = O.page_meta_batch(x["k"], x["sl"])
        r = O.route_pack_batch(x["v"], x["sc"], x["cls"], w.n_groups, w.k_nominal, w.t_cache * w.n_groups,
                               x["sl"])
        if w.token_budget is None:
            ids = n = None
        else:
            ids, n = O.select_batch(x["q"], kmin, kmax, w.token_budget, w.t_cache, x["sl"])
        O.attend_batch(x["q"], x["k"], w.n_groups, r["mask"], ids, n, SM_SCALE, packed=r["packed"],
                       offs=r["offs"], seq_len=x["sl"])
    dt = time.perf_counter() - t0
    return dict(seconds=dt)


def cpu_inputs(w: W.Workload, d: dict) -> dict:
    import oracle as O
    out = dict(k=O.bf16_bits(d["k"].cpu()), v=O.bf16_bits(d["v"].cpu()), q=O.bf16_bits(d["q"].cpu()),
               scores=d["scores"].cpu().numpy(),
               tok_class=None if d["tok_class"] is None else d["tok_class"].cpu().numpy(),
               seq_len=d["seq_len"].cpu().numpy())
    return out


# ------------------------------------------------------------------------ GPU arm
def select_workload(args) -> W.Workload:
    over = {}
    if args.budget is not None:
        over["token_budget"] = args.budget
    if args.keep is not None:
        over["k_nominal"] = args.keep
    if args.batch is not None:
        over["batch"] = args.batch
    if args.context is not None:
        over["t_cache"] = args.context
    return W.get(args.workload, **over)


def sample_problems(w: W.Workload, n: int):
    allp = [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]
    if n >= len(allp):
        return allp
    stride = len(allp) / n
    return [allp[int(i * stride)] for i in range(n)]


def run_gpu(args, r: D.Rank):
    import paper_2604_21335_b200 as P
    from paper_2604_21335_b200 import binding as Bd
    dev = torch.device("cuda", r.local_rank if r.world > 1 else 0)
    torch.cuda.set_device(dev)
    P.load_library()                       # fails loudly if the CUDA library is missing
    w = select_workload(args)
    w = W.shrink(w, seed=w.seed + 7919 * r.rank)          # each rank owns its own batch (weak scaling)
    NQ = 8
    d = W.make_inputs(w, dev, n_queries=NQ)
    B, Hkv, Hq, T, S = w.batch, w.n_kv_heads, w.n_q_heads, w.t_cache, w.n_groups
    shape = P.Shape(B, Hq, Hkv, S, T, d["seq_len"])
    n_full_tokens = w.n_text
    cap = (T - n_full_tokens) * w.k_nominal + n_full_tokens * S
    cache = P.Cache.allocate(shape, d["k"], cap)
    total = torch.zeros(B, Hkv, dtype=torch.int64, device=dev)
    status = torch.zeros(B, Hkv, dtype=torch.int32, device=dev)
    out = torch.zeros(B, Hq, 128, dtype=torch.float32, device=dev)
    if w.token_budget is None:
        page_ids = n_pages = None
        max_pages = shape.n_pages
    else:
        max_pages = max(1, min(shape.n_pages, w.token_budget // 16))
        page_ids = torch.zeros(B, Hkv, max_pages, dtype=torch.int32, device=dev)
        n_pages = torch.zeros(B, Hkv, dtype=torch.int32, device=dev)
    ws_r = Bd.new_workspace(shape, Bd.OP_ROUTE_PACK, device=dev)
    ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=dev)
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, max_pages, device=dev)
    qs = [d["q"][i].contiguous() for i in range(NQ)]
    names = ["page_meta", "route_mask", "pack_values", "quest_select", "decode_attn"]
    launches_per_step = 1 + 2 + (1 if page_ids is not None else 0) + 1   # route_pack = select kernel + compact kernel

    # The key side (page metadata, page selection) and the value side (routing, packing) of a
    # pass touch disjoint data, so they run on two streams and join before the attention call;
    # --serial puts all five calls on one stream.
    side = None if args.serial else torch.cuda.Stream(device=dev)

    def value_side():
        P.route_mask(shape, d["scores"], d["tok_class"], w.k_nominal, cache, ws_r)     # stc_route_pack, first half
        P.pack_values(shape, d["v"], cache, total, status, ws_r)                       # ... second half

    def step(i):
        q = qs[i % NQ]
        main = torch.cuda.current_stream()
        if side is not None:
            side.wait_stream(main)
            with torch.cuda.stream(side):
                value_side()
        P.build_page_meta(shape, cache)
        if side is None:
            value_side()
        if page_ids is not None:
            P.quest_select(shape, cache, q, w.token_budget, page_ids, n_pages, ws_s)
        if side is not None:
            main.wait_stream(side)
        P.decode_attn(shape, cache, q, page_ids, n_pages, SM_SCALE, out, ws_a)

    W_ = max(args.warmup, 3)
    for i in range(W_):
        step(i)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0, "device status reported an error"
    assert int(ws_a[:4].view(torch.int32)[0]) == 0, "stc_decode_attn device status"

    # algorithmic bytes from what the step actually kept / selected
    seq = d["seq_len"].cpu().tolist()
    cnt = torch.zeros_like(cache.v_mask, dtype=torch.int32)
    for j in range(S):
        cnt += (cache.v_mask.int() >> j) & 1
    if page_ids is not None:
        tok_idx = (page_ids.long()[..., None] * 16 + torch.arange(16, device=dev)).flatten(2)
        valid = tok_idx < d["seq_len"].long()[:, None, None]
        sel_groups = int((torch.gather(cnt, 2, tok_idx.clamp(max=T - 1)) * valid).sum())
        sel_tokens, sel_pages = int(valid.sum()), int(n_pages.sum())
    else:
        sel_groups, sel_tokens = int(cnt.sum()), int(sum(seq)) * Hkv
        sel_pages = int(sum((n + 15) // 16 for n in seq)) * Hkv
    del cnt
    n_routed = (int(sum(seq)) - n_full_tokens * B) * Hkv
    ab = algorithmic_bytes(w, seq, n_routed, n_full_tokens * B * Hkv, int(total.sum()), sel_pages,
                           sel_tokens, sel_groups)
    step_bytes = sum(ab.values())

    # ---- one CUDA graph per query set: a step is one graph launch, so the timed region holds
    #      device work only (a Python-driven launch sequence is CPU-bound on the small workloads)
    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    launch_mode = "cuda_graph"
    try:
        step_graphs = [capture(lambda j=j: step(j)) for j in range(NQ)]
        run_step = lambda i: step_graphs[i % NQ].replay()
    except Exception as e:                                   # noqa: BLE001
        if r.is_main:
            print(f"# graph capture unavailable ({type(e).__name__}: {e}); timing eager launches", file=sys.stderr)
        launch_mode = "eager"
        run_step = step
    for i in range(W_):
        run_step(i)
    torch.cuda.synchronize()

    # ---- timed region: exactly K steps -----------------------------------------------------------
    K = args.steps
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(dev.index or 0)
    D.barrier(r)
    torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for i in range(K):
        run_step(i)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    D.barrier(r)
    total_ms = D.max_over_ranks(r, ev0.elapsed_time(ev1))
    ms_per_step = total_ms / K
    value = step_bytes * r.world / (ms_per_step * 1e-3) / 1e9

    # ---- each call on its own: NQ back-to-back launches (rotating queries) per graph replay -------
    def call_fn(c, j):
        q = qs[j]
        if c == 0:
            P.build_page_meta(shape, cache)
        elif c == 1:
            P.route_mask(shape, d["scores"], d["tok_class"], w.k_nominal, cache, ws_r)
        elif c == 2:
            P.pack_values(shape, d["v"], cache, total, status, ws_r)
        elif c == 3:
            if page_ids is not None:
                P.quest_select(shape, cache, q, w.token_budget, page_ids, n_pages, ws_s)
        else:
            P.decode_attn(shape, cache, q, page_ids, n_pages, SM_SCALE, out, ws_a)

    per_call_ms = []
    for c in range(5):
        if c == 3 and page_ids is None:
            per_call_ms.append(0.0)
            continue
        body = lambda c=c: [call_fn(c, j) for j in range(NQ)]
        if launch_mode == "cuda_graph":
            g = capture(body)
            run = g.replay
        else:
            run = body
        run()
        torch.cuda.synchronize()
        reps = max(2, min(50, int(20.0 / max(ms_per_step * NQ, 1e-3))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        per_call_ms.append(e0.elapsed_time(e1) / (reps * NQ))
    if page_ids is not None:                                  # the last select ran with query NQ-1: redo the step's
        step(0)
        torch.cuda.synchronize()

    # ---- end to end through the C-ABI with host buffers ----------------------------
    e2e = None
    if not args.no_e2e:
        hk = d["k"].cpu().pin_memory(); hv = d["v"].cpu().pin_memory()
        hs = d["scores"].cpu().pin_memory()
        hc = None if d["tok_class"] is None else d["tok_class"].cpu().pin_memory()
        hq = [q.cpu().pin_memory() for q in qs]
        h_out = torch.zeros(B, Hq, 128, dtype=torch.float32).pin_memory()
        h_tot = torch.zeros(B, Hkv, dtype=torch.int64).pin_memory()
        h_st = torch.zeros(B, Hkv, dtype=torch.int32).pin_memory()
        arena = torch.empty(Bd.pass_host_arena_bytes(shape, cap, w.token_budget), dtype=torch.uint8, device=dev)
        Ke = max(1, min(K, args.e2e_steps))

        def e2e_step(i):
            Bd.pass_host(shape, hk, hv, hs, hc, hq[i % NQ], w.token_budget, w.k_nominal, SM_SCALE, cap,
                         arena, h_out, h_tot, h_st)
            torch.cuda.current_stream().synchronize()      # the step's result is read on the host
            return float(h_out[0, 0, 0])

        for i in range(2):
            e2e_step(i)
        D.barrier(r)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(Ke):
            e2e_step(i)
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / Ke
        e2e_ms = D.max_over_ranks(r, e2e_ms)
        assert int(h_st.abs().sum()) == 0
        # same result as the device-resident path (same query as the last timed step there)
        h2d = hk.numel() * 2 + hv.numel() * 2 + hs.numel() * 4 + (0 if hc is None else hc.numel()) + hq[0].numel() * 2
        d2h = h_out.numel() * 4 + h_tot.numel() * 8 + h_st.numel() * 4
        e2e = {"value": step_bytes * r.world / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": Ke, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        del hk, hv, hs, arena

    if not r.is_main:
        return
    peak, peak_src = peaks()
    per_kernel = {}
    for c, n in enumerate(names):
        ms = per_call_ms[c]
        gbs = ab[n] / (ms * 1e-3) / 1e9 if ms > 0 and ab[n] else 0.0
        per_kernel[n] = {"us": round(ms * 1e3, 2), "alg_bytes": ab[n], "GBps": round(gbs, 1),
                         "frac_of_" + peak_src: round(gbs / peak, 4), "frac_of_8TBps": round(gbs / NOMINAL_HBM_GBS, 4)}
    read_ms = per_call_ms[3] + per_call_ms[4]
    read_bytes = ab["quest_select"] + ab["decode_attn"]
    read_gbs = read_bytes / (read_ms * 1e-3) / 1e9
    # dominant call of the step (every call is one kernel)
    single = {n: per_call_ms[c] for c, n in enumerate(names) if ab[n]}
    dom = max(single, key=single.get)
    kernel_of = dict(KERNEL_OF)
    if (T + 255) // 256 <= 32 // S:                      # problems that fit one CTA take the small selection kernel
        kernel_of["route_mask"] = "route_select_small_kernel"
    roof = {"bound": "hbm", "kernel": kernel_of[dom], "achieved": per_kernel[dom]["GBps"], "peak": peak, "unit": UNIT,
            "frac": round(per_kernel[dom]["GBps"] / peak, 4), "peak_source": peak_src + " copy bandwidth",
            "traffic": TRAFFIC_NOTE.get((args.workload, dom))}
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": r.world, "steps": K,
        "warmup": W_, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{w.name}: B{B} Hq{Hq} Hkv{Hkv} T{T} S{S} keep{w.k_nominal} "
                               f"budget{w.token_budget}, one full pass per step "
                               "(page_meta + route_pack + quest_select + decode_attn)",
                   "l2": "inputs larger than L2 (K+V %.0f MiB re-read every step), %d rotating query sets"
                         % ((d["k"].numel() + d["v"].numel()) * 2 / 2 ** 20, NQ),
                   "replicas": "one independent batch per rank, no collective",
                   "streams": "one" if args.serial else "two (key side | value side, joined before decode_attn)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * K, "launch": launch_mode,
        "roofline": roof,
        "per_call": per_kernel,
        "read_side": {"us": round(read_ms * 1e3, 2), "alg_bytes": read_bytes, "GBps": round(read_gbs, 1),
                      "frac_of_" + peak_src: round(read_gbs / peak, 4),
                      "frac_of_8TBps": round(read_gbs / NOMINAL_HBM_GBS, 4)},
        "tokens_heads_per_s": {"context": round(B * Hq * T * r.world / (ms_per_step * 1e-3)),
                               "attended": round(sel_tokens * w.gq * r.world / (ms_per_step * 1e-3))},
    }
    if r.world == 1 and not args.no_cpu:
        dc = cpu_inputs(w, d)
        probs = sample_problems(w, args.cpu_problems)
        import oracle as O
        oracle_step(w, dc, probs[:1])                          # page in the library
        res = oracle_step(w, dc, probs)
        frac = len(probs) / w.n_problems
        line["cpu_baseline"] = {"value": round(step_bytes * frac / res["seconds"] / 1e9, 4), "unit": UNIT,
                                "cores": O.n_threads(), "kind": "oracle",
                                "sample": f"one full pass over {len(probs)} of {w.n_problems} (batch, kv head) "
                                          f"problems, {res['seconds']:.2f} s",
                                "tokens_heads_per_s_context": round(len(probs) * w.gq * T / res["seconds"])}
    print(json.dumps(line), flush=True)


KERNEL_OF = {"page_meta": "page_meta_kernel", "quest_select": "quest_select_kernel",
             "decode_attn": "decode_attn_kernel", "pack_values": "route_compact_kernel",
             "route_mask": "route_select_kernel"}

# Per-launch DRAM traffic of the dominant kernel from the committed ncu capture
# (profiles/), in bytes; None until a capture exists for that workload.
TRAFFIC_NOTE: dict = {
    # route_compact_kernel on this very workload: dram__bytes_read 205.7 MB + dram__bytes_write 83.0 MB per launch
    # (profiles/traffic_bench_cfg1.md; part of the packed store is still in L2 when the kernel ends)
    ("cfg1", "pack_values"): 288.5e6,
}


# ------------------------------------------------------------------ router (a "next" row)
D_MODEL = {"cfg2": 3584}                                    # Qwen2.5-7B; the other shapes are 4096-wide models


def run_router(args):
    """Times stc_router_logits alone on the workload's shape (not part of the step) and prints one line."""
    import paper_2604_21335_b200 as P
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = select_workload(args)
    B, T, Hkv, S = w.batch, w.t_cache, w.n_kv_heads, w.n_groups
    dm = D_MODEL.get(args.workload, 4096)
    g = torch.Generator(device=dev); g.manual_seed(w.seed ^ 0x707)
    NH = 2 if B * T * dm * 2 > (8 << 30) else 4                # rotating hidden-state sets, all larger than L2
    hs = [torch.randn(B, T, dm, generator=g, device=dev).to(torch.bfloat16) for _ in range(NH)]
    wt = (torch.randn(Hkv * S, dm, generator=g, device=dev) / dm ** 0.5).to(torch.bfloat16)
    sc = torch.empty(B, Hkv, T, S, dtype=torch.float32, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    shape = P.Shape(B, Hkv, Hkv, S, T)
    for i in range(max(args.warmup, 3)):
        P.router_logits(shape, hs[i % NH], wt, sc, st)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    K = args.steps
    e0.record()
    for i in range(K):
        P.router_logits(shape, hs[i % NH], wt, sc, st)
    e1.record()
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    us = e0.elapsed_time(e1) * 1e3 / K
    M, N = B * T, Hkv * S
    flops, nbytes = 2.0 * M * N * dm, M * dm * 2 + N * dm * 2 + M * N * 4
    peak_gbs, src = peaks()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak_tf = float(json.load(f)["bf16_tflops"])
    except Exception:
        peak_tf = 1590.0
    tf, gbs = flops / us / 1e6, nbytes / us / 1e3
    bound = "hbm" if nbytes / peak_gbs > flops / (peak_tf * 1e3) else "tensor"
    print(json.dumps({
        "metric": "router_logits", "us": round(us, 2), "TFLOPs": round(tf, 1), "GBps": round(gbs, 1),
        "config": {"workload": f"{w.name}: tokens {M}, logits {N}, d_model {dm}"},
        "roofline": {"bound": bound, "achieved": round(gbs if bound == "hbm" else tf, 1),
                     "peak": peak_gbs if bound == "hbm" else peak_tf, "unit": "GB/s" if bound == "hbm" else "TFLOP/s",
                     "frac": round((gbs / peak_gbs) if bound == "hbm" else (tf / peak_tf), 4),
                     "peak_source": src, "traffic": None},
        "steps": K, "data": "synthetic", "dtype": "bf16"}), flush=True)


# -------------------------------------------------------------------- reference arm
def run_reference(args, r: D.Rank):
    if not r.is_main:
        return
    import oracle as O
    w = select_workload(args)
    d = W.make_inputs(w, "cpu", n_queries=8)
    dc = cpu_inputs(w, d)
    probs = sample_problems(w, args.cpu_problems)
    frac = len(probs) / w.n_problems
    seq = dc["seq_len"].tolist()
    # bytes of the sample, with the selected / kept counts the configuration implies
    n_full = w.n_text
    n_routed = (sum(seq) - n_full * w.batch) * w.n_kv_heads
    total_groups = n_routed * w.k_nominal + n_full * w.batch * w.n_kv_heads * w.n_groups
    pages = sum((n + 15) // 16 for n in seq) * w.n_kv_heads
    if w.token_budget is None:
        sel_pages, sel_tokens = pages, sum(seq) * w.n_kv_heads
    else:
        sel_pages = min(w.token_budget // 16, (w.t_cache + 15) // 16) * w.n_problems
        sel_tokens = sel_pages * 16
    sel_groups = int(sel_tokens * total_groups / max(1, sum(seq) * w.n_kv_heads))
    ab = algorithmic_bytes(w, seq, n_routed, 0, total_groups, sel_pages, sel_tokens, sel_groups)
    step_bytes = sum(ab.values()) * frac
    for i in range(max(args.warmup, 1)):
        oracle_step(w, dc, probs[:max(1, len(probs) // 4)], i % 8)
    K = args.steps
    t0 = time.perf_counter()
    for i in range(K):
        oracle_step(w, dc, probs, i % 8)
    sec = (time.perf_counter() - t0) / K
    value = step_bytes / sec / 1e9
    sample = f"one full pass over {len(probs)} of {w.n_problems} (batch, kv head) problems per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": max(args.warmup, 1), "ms_per_step": round(sec * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name}: B{w.batch} Hq{w.n_q_heads} Hkv{w.n_kv_heads} T{w.t_cache} "
                               f"S{w.n_groups} keep{w.k_nominal} budget{w.token_budget}, CPU checker"},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": O.n_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1", choices=sorted(W.CONFIGS))
    ap.add_argument("--budget", type=int, default=None, help="override the Quest token budget")
    ap.add_argument("--keep", type=int, default=None, help="override the average groups kept")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--context", type=int, default=None)
    ap.add_argument("--cpu-problems", type=int, default=None, help="problems in the CPU-checker sample")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--serial", action="store_true", help="all calls of a step on one stream")
    ap.add_argument("--only", default=None, choices=["router"], help="time one extra kernel instead of the step")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        if args.cpu_problems is None:
            args.cpu_problems = 32
        world = int(os.environ.get("WORLD_SIZE", "1"))
        rank = int(os.environ.get("RANK", "0"))
        if world > 1 and rank != 0:
            return                                           # rank 0 alone runs the CPU arm
        run_reference(args, D.Rank())
        return
    if args.only == "router":
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        run_router(args)
        return
    args.steps = 300 if args.steps is None else args.steps
    args.warmup = 5 if args.warmup is None else args.warmup
    if args.cpu_problems is None:
        args.cpu_problems = 32
    r = D.init_from_env()
    try:
        run_gpu(args, r)
    finally:
        D.shutdown(r)


if __name__ == "__main__":
    main()
