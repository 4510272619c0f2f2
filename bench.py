#!/usr/bin/env python
"""Benchmark of the sub-token-routed decode path on B200.

One "step" is one decode step over a resident compressed cache:
  stc_quest_select -> stc_decode_attn
(query-aware page selection, then routed attention over the selected pages), on
synthetic inputs of the named workload; the write side (stc_build_page_meta,
stc_route_pack) builds that cache before the timed region and is reported on its
own (`per_call`, `full_pass`).  The metric is decode-attention GB/s: ALGORITHMIC
bytes of the step (page metadata scanned, selected keys, packed value groups,
masks, offsets, page ids, queries and outputs) divided by device time (CUDA
events around K graph replays with rotating query sets).  Every call is also
timed on its own, and `roofline` holds the dominant kernel of the step against
the measured copy bandwidth.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4]
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
FALLBACK_HBM_GBS = 6650.0        # used only when MEASURED_PEAKS.json is absent
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
class OracleSample:
    """The CPU checker on a sample of (batch, kv head) problems, laid out as a batch of
    one-KV-head sequences.  prepare() runs its write side once (untimed: it is not part of a decode
    step); read_step() is one decode step (page selection + routed attention) and is what is timed."""

    def __init__(self, w: W.Workload, d_cpu: dict, n_problems: int):
        import numpy as np
        import oracle as O
        self.O, self.np = O, np
        self.w = W.problem_view(w, list(range(n_problems)))      # batch = sample size, one KV head each
        self.full = w
        self.k, self.v = O.bf16_bits(d_cpu["k"]), O.bf16_bits(d_cpu["v"])
        self.q = O.bf16_bits(d_cpu["q"])                           # [NQ, n, Gq, 128]
        self.scores = d_cpu["scores"].numpy()
        self.cls = None if d_cpu["tok_class"] is None else d_cpu["tok_class"].numpy()
        self.seq_len = d_cpu["seq_len"].numpy()
        self.state = None

    def prepare(self):
        O, w = self.O, self.full
        kmin, kmax = O.page_meta_batch(self.k, self.seq_len)
        r = O.route_pack_batch(self.v, self.scores, self.cls, w.n_groups, w.k_nominal,
                               w.t_cache * w.n_groups, self.seq_len)
        self.state = dict(kmin=kmin, kmax=kmax, **r)

    def read_step(self, qi: int):
        O, w, st = self.O, self.full, self.state
        t0 = time.perf_counter()
        if w.token_budget is None:
            ids = n = None
        else:
            ids, n = O.select_batch(self.q[qi], st["kmin"], st["kmax"], w.token_budget, w.t_cache, self.seq_len)
        out, lse = O.attend_batch(self.q[qi], self.k, w.n_groups, st["mask"], ids, n, SM_SCALE,
                                  packed=st["packed"], offs=st["offs"], seq_len=self.seq_len)
        return time.perf_counter() - t0, out, ids, n

    def near_ties(self, qi: int, rel: float = 1e-6) -> int:
        """Pages whose fp64 bound lies within rel*max(1,|U_k|) of the k-th largest, summed over the sample."""
        w, st = self.full, self.state
        if w.token_budget is None:
            return 0
        return int(self.O.near_ties_batch(self.q[qi], st["kmin"], st["kmax"], w.token_budget, w.t_cache,
                                          self.seq_len, rel).sum())


def sample_bytes(w: W.Workload, n_problems: int, ab_read: int) -> float:
    return ab_read * n_problems / w.n_problems


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


def workload_string(w: W.Workload) -> str:
    return (f"{w.name}: B{w.batch} Hq{w.n_q_heads} Hkv{w.n_kv_heads} T{w.t_cache} S{w.n_groups} "
            f"keep{w.k_nominal} budget{w.token_budget}, one decode step per step "
            "(stc_quest_select + stc_decode_attn over the resident compressed cache)")     # = stc_decode_step


L2_BYTES = 126 << 20
NQ = 8                                                      # rotating query sets


def read_bytes_estimate(w: W.Workload) -> int:
    """Shape-only estimate of a decode step's algorithmic bytes (sizes the number of cache copies)."""
    sel = w.n_pages if w.token_budget is None else min(w.n_pages, w.token_budget // 16)
    per = sel * 16 * (256 + w.k_nominal * w.group_dim * 2 + 2)
    if w.token_budget is not None:
        per += w.n_pages * 512
    return per * w.n_problems


class Copy:
    """One resident cache (inputs, compressed store, write-side workspaces)."""

    def __init__(self, P, Bd, w, dev, seed):
        self.w = W.shrink(w, seed=seed)
        self.d = W.make_inputs(self.w, dev, n_queries=NQ)
        B, Hkv, Hq, T, S = w.batch, w.n_kv_heads, w.n_q_heads, w.t_cache, w.n_groups
        self.shape = P.Shape(B, Hq, Hkv, S, T, self.d["seq_len"])
        self.cap = (T - w.n_text) * w.k_nominal + w.n_text * S
        self.cache = P.Cache.allocate(self.shape, self.d["k"], self.cap)
        self.total = torch.zeros(B, Hkv, dtype=torch.int64, device=dev)
        self.status = torch.zeros(B, Hkv, dtype=torch.int32, device=dev)
        self.ws_r = Bd.new_workspace(self.shape, Bd.OP_ROUTE_PACK, device=dev)
        self.qs = [self.d["q"][i].contiguous() for i in range(NQ)]


def run_gpu(args, r: D.Rank):
    import paper_2604_21335_b200 as P
    from paper_2604_21335_b200 import binding as Bd
    dev = torch.device("cuda", r.local_rank if r.world > 1 else 0)
    torch.cuda.set_device(dev)
    P.load_library()                       # fails loudly if the CUDA library is missing
    w = select_workload(args)
    B, Hkv, Hq, T, S = w.batch, w.n_kv_heads, w.n_q_heads, w.t_cache, w.n_groups
    # Decode steps whose working set fits L2 would be served from L2 by the second step: such
    # workloads rotate independent cache copies (one per query set) so that consecutive steps
    # touch different lines; larger ones use one cache and rotate the queries only.
    n_copies = 1 if read_bytes_estimate(w) >= 2 * L2_BYTES else NQ
    copies = [Copy(P, Bd, w, dev, w.seed + 7919 * r.rank + 104729 * c) for c in range(n_copies)]
    shape = copies[0].shape
    if w.token_budget is None:
        max_pages = shape.n_pages
        ids = npg = [None] * NQ
    else:
        max_pages = max(1, min(shape.n_pages, w.token_budget // 16))
        ids = [torch.zeros(B, Hkv, max_pages, dtype=torch.int32, device=dev) for _ in range(NQ)]
        npg = [torch.zeros(B, Hkv, dtype=torch.int32, device=dev) for _ in range(NQ)]
    out = torch.zeros(B, Hq, 128, dtype=torch.float32, device=dev)
    ws_s = Bd.new_workspace(shape, Bd.OP_QUEST_SELECT, device=dev)
    ws_a = Bd.new_workspace(shape, Bd.OP_DECODE_ATTN, max_pages, device=dev)
    names = ["page_meta", "route_mask", "pack_values", "quest_select", "decode_attn"]
    side = None if args.serial else torch.cuda.Stream(device=dev)

    def copy_of(j):
        return copies[j % n_copies]

    def value_side(c):
        P.route_mask(c.shape, c.d["scores"], c.d["tok_class"], w.k_nominal, c.cache, c.ws_r)
        P.pack_values(c.shape, c.d["v"], c.cache, c.total, c.status, c.ws_r)

    def write_side(j):
        # the key side (page metadata) and the value side (routing, packing) touch disjoint data:
        # two streams, joined at the end; --serial keeps one stream
        c = copy_of(j)
        main = torch.cuda.current_stream()
        if side is not None:
            side.wait_stream(main)
            with torch.cuda.stream(side):
                value_side(c)
        P.build_page_meta(c.shape, c.cache)
        if side is None:
            value_side(c)
        else:
            main.wait_stream(side)

    def read_step(j):
        c = copy_of(j)
        if ids[j] is not None and not args.two_calls:
            # stc_decode_step = stc_quest_select + stc_decode_attn as one call
            P.decode_step(c.shape, c.cache, c.qs[j], w.token_budget, ids[j], npg[j], SM_SCALE, out, ws_s, ws_a)
            return
        if ids[j] is not None:
            P.quest_select(c.shape, c.cache, c.qs[j], w.token_budget, ids[j], npg[j], ws_s)
        P.decode_attn(c.shape, c.cache, c.qs[j], ids[j], npg[j], SM_SCALE, out, ws_a)

    # ---- build the resident caches (the write side; also its warm-up), then warm the read side --
    W_ = max(args.warmup, 3)
    for c in range(n_copies):
        write_side(c)
    for i in range(max(W_, NQ)):
        read_step(i % NQ)
    torch.cuda.synchronize()
    for c in copies:
        assert int(c.status.abs().sum()) == 0, "device status reported an error"
    assert int(ws_a[:4].view(torch.int32)[0]) == 0, "stc_decode_attn device status"

    # ---- algorithmic bytes from what the steps actually kept / selected (mean over the query sets)
    seq = copies[0].d["seq_len"].cpu().tolist()
    n_routed = (int(sum(seq)) - w.n_text * B) * Hkv
    abs_ = []
    for j in range(NQ):
        c = copy_of(j)
        cnt = torch.zeros_like(c.cache.v_mask, dtype=torch.int32)
        for g_ in range(S):
            cnt += (c.cache.v_mask.int() >> g_) & 1
        if ids[j] is not None:
            tok_idx = (ids[j].long()[..., None] * 16 + torch.arange(16, device=dev)).flatten(2)
            valid = tok_idx < c.d["seq_len"].long()[:, None, None]
            sel_groups = int((torch.gather(cnt, 2, tok_idx.clamp(max=T - 1)) * valid).sum())
            sel_tokens, sel_pages = int(valid.sum()), int(npg[j].sum())
        else:
            sel_groups, sel_tokens = int(cnt.sum()), int(sum(seq)) * Hkv
            sel_pages = int(sum((n + 15) // 16 for n in seq)) * Hkv
        del cnt
        abs_.append((algorithmic_bytes(w, seq, n_routed, w.n_text * B * Hkv, int(c.total.sum()), sel_pages,
                                       sel_tokens, sel_groups), sel_tokens))
    ab = {n: sum(a[n] for a, _ in abs_) // NQ for n in names}
    sel_tokens = sum(t for _, t in abs_) // NQ
    read_bytes = ab["quest_select"] + ab["decode_attn"]
    pass_bytes = sum(ab.values())

    # ---- one CUDA graph per query set: a step is one graph launch, so the timed region holds
    #      device work only (a Python-driven launch sequence is CPU-bound on the small workloads)
    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g

    launch_mode = "cuda_graph"
    try:
        step_graphs = [capture(lambda j=j: read_step(j)) for j in range(NQ)]
        run_step = lambda i: step_graphs[i % NQ].replay()
    except Exception as e:                                   # noqa: BLE001
        if r.is_main:
            print(f"# graph capture unavailable ({type(e).__name__}: {e}); timing eager launches", file=sys.stderr)
        launch_mode = "eager"
        run_step = lambda i: read_step(i % NQ)
    for i in range(max(W_, NQ)):
        run_step(i)
    torch.cuda.synchronize()

    # ---- timed region: exactly K decode steps ----------------------------------------------------
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
    value = read_bytes * r.world / (ms_per_step * 1e-3) / 1e9

    def timed(run, reps):
        run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def graphed(body):
        if launch_mode == "cuda_graph":
            return capture(body).replay
        return body

    # ---- each call on its own: NQ back-to-back launches per graph replay, query set j on its own
    #      cache copy and (decode_attn) with the page list that query selected ------------------------
    def call_fn(cidx, j):
        c = copy_of(j)
        if cidx == 0:
            P.build_page_meta(c.shape, c.cache)
        elif cidx == 1:
            P.route_mask(c.shape, c.d["scores"], c.d["tok_class"], w.k_nominal, c.cache, c.ws_r)
        elif cidx == 2:
            P.pack_values(c.shape, c.d["v"], c.cache, c.total, c.status, c.ws_r)
        elif cidx == 3:
            P.quest_select(c.shape, c.cache, c.qs[j], w.token_budget, ids[j], npg[j], ws_s)
        else:
            P.decode_attn(c.shape, c.cache, c.qs[j], ids[j], npg[j], SM_SCALE, out, ws_a)

    budget_ms = 400.0                                        # device time spent on each extra measurement
    per_call_ms = []
    for cidx in range(5):
        if cidx == 3 and ids[0] is None:
            per_call_ms.append(0.0)
            continue
        run = graphed(lambda cidx=cidx: [call_fn(cidx, j) for j in range(NQ)])
        est = ms_per_step * NQ * (8.0 if cidx < 3 else 1.0)
        per_call_ms.append(timed(run, max(2, min(50, int(budget_ms / max(est, 1e-3))))) / NQ)

    # ---- the whole pass (write side + decode step), as an extra figure ---------------------------
    run = graphed(lambda: [(write_side(j), read_step(j)) for j in range(NQ)])
    pass_ms = timed(run, max(1, min(20, int(budget_ms / max(sum(per_call_ms) * NQ, 1e-3))))) / NQ
    torch.cuda.synchronize()
    for c in copies:
        assert int(c.status.abs().sum()) == 0

    # ---- the write side from hidden states: router logits (tcgen05 GEMM) -> masks -> packed store ----
    write_from_hidden = None
    if not args.no_router and (Hkv * S <= 256 or (Hkv * S) % 256 == 0):
        c0 = copies[0]
        dm = D_MODEL.get(w.name.split("x")[0], 4096)
        gen = torch.Generator(device=dev); gen.manual_seed(w.seed ^ 0x707)
        hs = torch.empty(B, T, dm, dtype=torch.bfloat16, device=dev)
        for b in range(B):
            hs[b] = torch.randn(T, dm, generator=gen, device=dev).to(torch.bfloat16)
        wt = (torch.randn(Hkv * S, dm, generator=gen, device=dev) / dm ** 0.5).to(torch.bfloat16)
        sc2 = torch.empty(B, Hkv, T, S, dtype=torch.float32, device=dev)
        st_word = torch.zeros(1, dtype=torch.int32, device=dev)
        cache2 = P.Cache.allocate(c0.shape, c0.d["k"], T * S if w.n_text else c0.cap)
        tot2, stat2 = torch.zeros_like(c0.total), torch.zeros_like(c0.status)

        def from_hidden():
            P.router_logits(c0.shape, hs, wt, sc2, st_word)
            P.route_mask(c0.shape, sc2, c0.d["tok_class"], w.k_nominal, cache2, c0.ws_r)
            P.pack_values(c0.shape, c0.d["v"], cache2, tot2, stat2, c0.ws_r)

        t_all = timed(graphed(from_hidden), max(2, min(20, int(budget_ms / max(sum(per_call_ms[1:3]) * 2, 1e-3)))))
        t_rt = timed(graphed(lambda: P.router_logits(c0.shape, hs, wt, sc2, st_word)),
                     max(2, min(20, int(budget_ms / max(per_call_ms[1], 1e-3)))))
        torch.cuda.synchronize()
        assert int(st_word[0]) == 0 and int(stat2.abs().sum()) == 0
        rt_bytes = B * T * dm * 2 + Hkv * S * dm * 2 + B * T * Hkv * S * 4
        write_from_hidden = {"us": round(t_all * 1e3, 2), "router_logits_us": round(t_rt * 1e3, 2),
                             "router_logits_GBps": round(rt_bytes / (t_rt * 1e-3) / 1e9, 1),
                             "router_logits_TFLOPs": round(2.0 * B * T * Hkv * S * dm / (t_rt * 1e-3) / 1e12, 1),
                             "d_model": dm,
                             "calls": "stc_router_logits -> stc_route_mask -> stc_pack_values (synthetic router weights)"}
        del hs, sc2, cache2

    # ---- the CPU checker on a sample of problems: timed baseline, parity check, near-tie count ----
    probs = sample_problems(w, args.cpu_problems)
    cpu_baseline = checked = None
    oracle_out = None
    if r.world == 1 and not args.no_cpu:
        import numpy as np
        import oracle as O
        c0 = copies[0]
        d_cpu = dict(k=torch.stack([c0.d["k"][b, h:h + 1] for b, h in probs]).cpu(),
                     v=torch.stack([c0.d["v"][b, h:h + 1] for b, h in probs]).cpu(),
                     scores=torch.stack([c0.d["scores"][b, h:h + 1] for b, h in probs]).cpu(),
                     q=torch.stack([c0.d["q"][:, b, h * w.gq:(h + 1) * w.gq] for b, h in probs], dim=1).cpu(),
                     tok_class=None if c0.d["tok_class"] is None else
                     torch.stack([c0.d["tok_class"][b] for b, _ in probs]).cpu(),
                     seq_len=torch.stack([c0.d["seq_len"][b] for b, _ in probs]).cpu())
        smp = OracleSample(c0.w, d_cpu, len(probs))
        smp.prepare()
        smp.read_step(0)                                       # page in the library
        secs, oracle_out = 0.0, None
        for qi in range(NQ):
            if n_copies > 1 and qi > 0:
                break                                          # other query sets belong to other cache copies
            dt, o_out, o_ids, o_n = smp.read_step(qi)
            secs += dt
            if qi == 0:
                oracle_out, oracle_ids, oracle_n = o_out, o_ids, o_n
        n_steps_cpu = 1 if n_copies > 1 else NQ
        cpu_baseline = {"value": round(sample_bytes(w, len(probs), read_bytes) * n_steps_cpu / secs / 1e9, 4),
                        "unit": UNIT, "cores": O.n_threads(), "kind": "oracle",
                        "sample": f"{n_steps_cpu} decode step(s) over {len(probs)} of {w.n_problems} "
                                  f"(batch, kv head) problems, {secs:.2f} s (its write side, untimed, ran once)",
                        "tokens_heads_per_s_context": round(len(probs) * w.gq * T * n_steps_cpu / secs)}

        def sample_err(o_t):                                    # [B,Hq,128] tensor vs the checker's sample
            got = torch.stack([o_t[b, h * w.gq:(h + 1) * w.gq] for b, h in probs]).double().cpu().numpy()
            diff = np.abs(got - oracle_out)
            return float(diff.max()), float(diff.mean() / max(np.abs(oracle_out).mean(), 1e-30))

        read_step(0)
        torch.cuda.synchronize()
        ma, mr = sample_err(out)
        assert ma <= 1e-2 and mr <= 2e-3, ("device-resident decode step vs CPU checker", ma, mr)
        if ids[0] is not None:
            for i, (b, h) in enumerate(probs):
                assert int(npg[0][b, h]) == int(oracle_n[i, 0])
                assert np.array_equal(ids[0][b, h, :int(oracle_n[i, 0])].cpu().numpy(),
                                      oracle_ids[i, 0, :int(oracle_n[i, 0])]), "page ids differ from the CPU checker"
        checked = {"problems": len(probs), "page_ids": "bit-exact" if ids[0] is not None else "selection off",
                   "decode_step": {"max_abs": ma, "mean_rel": mr},
                   "near_tie_pages_1e-6": smp.near_ties(0)}

    # ---- end to end through the C-ABI with host buffers ----------------------------
    e2e = e2e_pass = None
    if not args.no_e2e:
        c0 = copies[0]
        hq = [q.cpu().pin_memory() for q in c0.qs]
        h_out = torch.zeros(B, Hq, 128, dtype=torch.float32).pin_memory()
        h_st = torch.full((1,), -1, dtype=torch.int32).pin_memory()
        arena = torch.empty(Bd.decode_step_host_arena_bytes(shape, w.token_budget), dtype=torch.uint8, device=dev)
        Ke = max(1, min(K, args.e2e_steps))

        def e2e_step(i):                                    # the cache stays resident; the query comes from the host
            Bd.decode_step_host(shape, c0.cache, hq[i % NQ], w.token_budget, SM_SCALE, arena, h_out, h_st)
            torch.cuda.current_stream().synchronize()      # the step's result is read on the host
            return float(h_out[0, 0, 0])

        e2e_step(0)
        assert int(h_st[0]) == 0
        if oracle_out is not None:                          # same result as the checker before anything is timed
            ma, mr = sample_err(h_out)
            assert ma <= 1e-2 and mr <= 2e-3, ("stc_decode_step_host vs CPU checker", ma, mr)
            checked["decode_step_host"] = {"max_abs": ma, "mean_rel": mr}
        for i in range(3):
            e2e_step(i)
        D.barrier(r)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(Ke):
            e2e_step(i)
        torch.cuda.synchronize()
        e2e_ms = D.max_over_ranks(r, (time.perf_counter() - t0) * 1e3 / Ke)
        e2e = {"value": read_bytes * r.world / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": Ke, "h2d_bytes_per_step": hq[0].numel() * 2, "d2h_bytes_per_step": h_out.numel() * 4 + 4,
               "call": "stc_decode_step_host (query from pinned host memory, selection + attention on the "
                       "resident cache, result back to the host)"}
        del arena

        if not args.no_e2e_pass:
            # the whole pass from host buffers (keys, values and scores cross PCIe every step)
            hk = c0.d["k"].cpu().pin_memory(); hv = c0.d["v"].cpu().pin_memory()
            hs = c0.d["scores"].cpu().pin_memory()
            hc = None if c0.d["tok_class"] is None else c0.d["tok_class"].cpu().pin_memory()
            h_tot = torch.zeros(B, Hkv, dtype=torch.int64).pin_memory()
            h_stp = torch.zeros(B, Hkv, dtype=torch.int32).pin_memory()
            arena = torch.empty(Bd.pass_host_arena_bytes(shape, c0.cap, w.token_budget), dtype=torch.uint8, device=dev)
            h2d = hk.numel() * 2 + hv.numel() * 2 + hs.numel() * 4 + (0 if hc is None else hc.numel()) + hq[0].numel() * 2
            Kp = max(1, min(Ke, int(2e10 // h2d) or 1, 20))

            def pass_step(i):
                Bd.pass_host(shape, hk, hv, hs, hc, hq[i % NQ], w.token_budget, w.k_nominal, SM_SCALE, c0.cap,
                             arena, h_out, h_tot, h_stp)
                torch.cuda.current_stream().synchronize()

            pass_step(0)
            assert int(h_stp.abs().sum()) == 0
            if oracle_out is not None:
                ma, mr = sample_err(h_out)
                assert ma <= 1e-2 and mr <= 2e-3, ("stc_pass_host vs CPU checker", ma, mr)
                checked["pass_host"] = {"max_abs": ma, "mean_rel": mr}
            t0 = time.perf_counter()
            for i in range(Kp):
                pass_step(i)
            torch.cuda.synchronize()
            p_ms = D.max_over_ranks(r, (time.perf_counter() - t0) * 1e3 / Kp)
            e2e_pass = {"value": pass_bytes * r.world / (p_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": p_ms,
                        "steps": Kp, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": h_out.numel() * 4 + h_tot.numel() * 8 + h_stp.numel() * 4,
                        "call": "stc_pass_host (whole pass from pinned host buffers)"}
            del hk, hv, hs, arena

    if not r.is_main:
        return
    peak, peak_src = peaks()
    per_kernel = {}
    for cidx, n in enumerate(names):
        ms = per_call_ms[cidx]
        gbs = ab[n] / (ms * 1e-3) / 1e9 if ms > 0 and ab[n] else 0.0
        per_kernel[n] = {"us": round(ms * 1e3, 2), "alg_bytes": ab[n], "GBps": round(gbs, 1),
                         "frac_of_" + peak_src: round(gbs / peak, 4), "frac_of_8TBps": round(gbs / NOMINAL_HBM_GBS, 4)}
    # dominant kernel of the timed step (each call of the step is one kernel)
    step_calls = {n: per_call_ms[names.index(n)] for n in ("quest_select", "decode_attn") if ab[n]}
    dom = max(step_calls, key=step_calls.get)
    traffic = TRAFFIC_NOTE.get((w.name, w.batch, w.token_budget, w.k_nominal, dom))
    sel_kernel = ("quest_filter_kernel" if (w.gq >= 2 and w.n_pages >= 4096) or (w.gq > 4 and w.n_pages >= 1024)
                  else "quest_select_kernel") + f"<{w.gq}>"      # the library's own choice of scan, restated
    roof = {"bound": "hbm", "kernel": sel_kernel if dom == "quest_select" else KERNEL_OF[dom],
            "achieved": per_kernel[dom]["GBps"], "peak": peak, "unit": UNIT,
            "frac": round(per_kernel[dom]["GBps"] / peak, 4), "peak_source": peak_src + " copy bandwidth",
            "traffic": traffic}
    ws_mib = read_bytes / 2 ** 20
    if n_copies == 1:
        l2 = ("a decode step moves %.0f MiB (larger than L2, page metadata re-read every step); %d rotating query "
              "sets, each with its own page list" % (ws_mib, NQ))
    else:
        l2 = ("a decode step moves %.0f MiB (fits L2): %d independent cache copies rotate with the query sets, so "
              "consecutive steps touch different lines (%.0f MiB per rotation)" % (ws_mib, n_copies, ws_mib * n_copies))
    if ws_mib * n_copies < 2 * L2_BYTES / 2 ** 20:
        l2 += "; L2-assisted: the rotation is smaller than twice L2"
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": r.world, "steps": K,
        "warmup": max(W_, NQ), "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_string(w), "l2": l2,
                   "replicas": "one independent batch per rank, no collective"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": (2 if ids[0] is not None else 1) * K, "launch": launch_mode,
        "roofline": roof,
        "frac_of_" + peak_src: round(value / r.world / peak, 4), "frac_of_8TBps": round(value / r.world / NOMINAL_HBM_GBS, 4),
        "per_call": per_kernel,
        "read_side": {"us": round(ms_per_step * 1e3, 2), "alg_bytes": read_bytes, "GBps": round(value / r.world, 1),
                      "sum_of_calls_us": round((per_call_ms[3] + per_call_ms[4]) * 1e3, 2)},
        "full_pass": {"us": round(pass_ms * 1e3, 2), "alg_bytes": pass_bytes,
                      "GBps": round(pass_bytes / (pass_ms * 1e-3) / 1e9, 1),
                      "streams": "one" if args.serial else "two (page metadata | routing + packing, joined before the decode step)"},
        "e2e_full_pass": e2e_pass,
        "write_side_from_hidden": write_from_hidden,
        "tokens_heads_per_s": {"context": round(B * Hq * T * r.world / (ms_per_step * 1e-3)),
                               "attended": round(sel_tokens * w.gq * r.world / (ms_per_step * 1e-3))},
    }
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
        line["checked_against_cpu"] = checked
    print(json.dumps(line), flush=True)


KERNEL_OF = {"page_meta": "page_meta_kernel", "quest_select": "quest_select_kernel",   # (or quest_filter_kernel, see below)
             "decode_attn": "decode_attn_kernel", "pack_values": "route_compact_kernel",
             "route_mask": "route_band_kernel"}   # (route_select_kernel below half the L2 size of scores; never the step's dominant call)

# Per-launch DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, bytes) of the step's dominant
# kernel from the committed ncu captures under profiles/, keyed by (workload, batch, budget, keep, call);
# absent = no capture of the kernel as it stands.
TRAFFIC_NOTE: dict = {
    # quest_filter_kernel<4>: dram__bytes_read 134.71 MB + dram__bytes_write 4.36 MB per launch at batch 4
    # (profiles/ncu_full_select_attn_cfg4_batch4.md), scaled by 4 to the 16 sequences of the full workload (the
    # traffic is the metadata scan plus the score array, both proportional to the number of problems)
    ("cfg4", 16, 4096, 4, "quest_select"): 4 * (134.71e6 + 4.36e6),
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
    """The CPU checker as it stands on a sample of the same workload: its write side once
    (untimed), then K decode steps (page selection + routed attention) with rotating queries."""
    if not r.is_main:
        return
    import oracle as O
    w = select_workload(args)
    probs = sample_problems(w, args.cpu_problems)
    d = W.make_inputs(w, "cpu", n_queries=NQ, problems=probs)       # the same bits the GPU arm draws
    smp = OracleSample(w, d, len(probs))
    smp.prepare()
    # bytes of the sample, with the selected / kept counts the configuration implies
    seq = [w.t_cache] * w.batch
    n_routed = (sum(seq) - w.n_text * w.batch) * w.n_kv_heads
    total_groups = n_routed * w.k_nominal + w.n_text * w.batch * w.n_kv_heads * w.n_groups
    pages = sum((n + 15) // 16 for n in seq) * w.n_kv_heads
    if w.token_budget is None:
        sel_pages, sel_tokens = pages, sum(seq) * w.n_kv_heads
    else:
        sel_pages = min(w.token_budget // 16, (w.t_cache + 15) // 16) * w.n_problems
        sel_tokens = sel_pages * 16
    sel_groups = int(sel_tokens * total_groups / max(1, sum(seq) * w.n_kv_heads))
    ab = algorithmic_bytes(w, seq, n_routed, 0, total_groups, sel_pages, sel_tokens, sel_groups)
    step_bytes = sample_bytes(w, len(probs), ab["quest_select"] + ab["decode_attn"])
    for i in range(max(args.warmup, 1)):
        smp.read_step(i % NQ)
    K = args.steps
    sec = sum(smp.read_step(i % NQ)[0] for i in range(K)) / K
    value = step_bytes / sec / 1e9
    sample = (f"one decode step over {len(probs)} of {w.n_problems} (batch, kv head) problems per step "
              "(its write side, untimed, ran once)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": max(args.warmup, 1), "ms_per_step": round(sec * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(w)},
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
    ap.add_argument("--workload", default="cfg4", choices=sorted(W.CONFIGS))
    ap.add_argument("--budget", type=int, default=None, help="override the Quest token budget")
    ap.add_argument("--keep", type=int, default=None, help="override the average groups kept")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--context", type=int, default=None)
    ap.add_argument("--cpu-problems", type=int, default=None, help="problems in the CPU-checker sample")
    ap.add_argument("--e2e-steps", type=int, default=100)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-e2e-pass", action="store_true", help="skip the whole pass from host buffers")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--two-calls", action="store_true",
                    help="time the decode step as stc_quest_select + stc_decode_attn instead of stc_decode_step")
    ap.add_argument("--no-router", action="store_true", help="skip the write side measured from hidden states")
    ap.add_argument("--serial", action="store_true", help="the write side of the full pass on one stream")
    ap.add_argument("--only", default=None, choices=["router"], help="time one extra kernel instead of the step")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 16 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        if args.cpu_problems is None:
            args.cpu_problems = 8
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
    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 8 if args.warmup is None else args.warmup
    if args.cpu_problems is None:
        args.cpu_problems = 16
    r = D.init_from_env()
    try:
        run_gpu(args, r)
    finally:
        D.shutdown(r)


if __name__ == "__main__":
    main()
