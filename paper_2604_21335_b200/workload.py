"""Seeded synthetic inputs shaped like the paper's decode workloads.

This module only draws random tensors and lays them out; it contains none of
the method's arithmetic (no page bounds, no selection, no routing, no
attention), so both the CUDA path and the CPU checker can be fed from it.

Shapes follow the paper's settings: LLaMA-2-7B-like multi-head attention,
Qwen2.5-7B-like grouped-query attention, a LLaVA-1.5-7B-like cache of 576
visual + text tokens reduced to a quarter of the visual tokens (Appendix
"Training Details and Implementation Cost", VLM paragraph), value groups
S in {8, 16} with K/S budgets from Section 3.3 / Appendix C.

Value recipe (all configs): Q, K, V iid N(0,1) (65536 equiprobable levels, counter-based, the same
bits on every device) rounded to bf16; in K, four
channels per KV head (ids drawn once per head from the seed) are multiplied
by 8 before rounding.  Router scores are fp32 per (batch, kv head, token,
group): iid N(0,1), or the L2 norm of the bf16 value group plus N(0, 0.5).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch

HEAD_DIM = 128
PAGE = 16

CLS_DROP, CLS_ROUTED, CLS_FULL = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    t_cache: int                 # cached tokens per sequence seen by the library
    n_groups: int                # S
    k_nominal: int               # average groups kept per routed token
    token_budget: Optional[int]  # Quest token budget; None = selection off
    score_recipe: str = "normal"  # "normal" | "vnorm"
    # VLM-style cache: leading text tokens keep full values, the rest are the
    # survivors of an upstream visual-token reducer (seeded random stand-in).
    n_text: int = 0
    n_visual_total: int = 0
    visual_keep: float = 1.0
    seed: int = 0x5C7C0000

    @property
    def gq(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_problems(self) -> int:
        return self.batch * self.n_kv_heads

    @property
    def n_pages(self) -> int:
        return (self.t_cache + PAGE - 1) // PAGE

    @property
    def group_dim(self) -> int:
        return HEAD_DIM // self.n_groups


def _vlm_cache_len(n_text: int, n_vis: int, keep: float) -> int:
    return n_text + int(round(n_vis * keep))


CONFIGS: Dict[str, Workload] = {
    # tiny MHA case the CPU checker finishes in seconds
    "cfg0": Workload("cfg0", 1, 8, 8, 4096, 8, 4, 1024, "normal", seed=0x5C7C0000),
    # LLaMA-2-7B-shaped, one layer
    "cfg1": Workload("cfg1", 1, 32, 32, 32768, 8, 4, 2048, "vnorm", seed=0x5C7C0001),
    # Qwen2.5-7B-shaped GQA (7 query heads per KV head)
    "cfg2": Workload("cfg2", 8, 28, 4, 32768, 16, 4, 4096, "normal", seed=0x5C7C0002),
    # LLaVA-1.5-7B-shaped cache: 128 text + 25% of 576 visual tokens
    "cfg3": Workload("cfg3", 32, 32, 32, _vlm_cache_len(128, 576, 0.25), 8, 3, None, "normal",
                     n_text=128, n_visual_total=576, visual_keep=0.25, seed=0x5C7C0003),
    # cfg1 for all 32 layers of the model in one call: the layers' caches are stacked along the
    # batch axis (the library treats every (batch, kv head) problem independently, so a stack
    # of layers is just a larger batch) -- amortises the per-call latency of the small configs
    "cfg1x32": Workload("cfg1x32", 32, 32, 32, 32768, 8, 4, 2048, "vnorm", seed=0x5C7C0011),
    # cfg2 for all 28 layers of the Qwen2.5-7B-shaped model in one call (7 query heads per KV head, S = 16)
    "cfg2x28": Workload("cfg2x28", 8 * 28, 28, 4, 32768, 16, 4, 4096, "normal", seed=0x5C7C0012),
    # long-context GQA sweep base point (budget / k_nominal overridden per point)
    "cfg4": Workload("cfg4", 16, 32, 8, 131072, 8, 4, 4096, "normal", seed=0x5C7C0004),
}

CFG4_BUDGETS = (256, 1024, 4096)
CFG4_KEEPS = (1, 2, 4, 8)


def get(name: str, **overrides) -> Workload:
    w = CONFIGS[name]
    return replace(w, **overrides) if overrides else w


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


# ---------------------------------------------------------------------------------------------
# Counter-based draws.  Every element of every tensor is a pure function of (seed, tensor id,
# problem index, element index): a 32-bit integer hash picks one of 65536 equiprobable levels of
# the standard normal (inverse CDF at the level's mid-point, tabulated once on the host in fp64).
# Only integer arithmetic follows the table, so the CPU and the GPU draw bit-identical tensors,
# and any subset of (batch, kv head) problems can be drawn without drawing the rest.
_T_K, _T_V, _T_SCORE, _T_Q = 1, 2, 3, 4
_M64 = (1 << 64) - 1
_TABLE = None


def _normal_table() -> torch.Tensor:
    global _TABLE
    if _TABLE is None:
        u = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _TABLE = (math.sqrt(2.0) * torch.special.erfinv(2.0 * u - 1.0)).to(torch.float32)
    return _TABLE


def _splitmix64(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _M64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


def _i32(x: int) -> int:
    x &= 0xFFFFFFFF
    return x - (1 << 32) if x >= (1 << 31) else x


def _keys(seed: int, tensor_id: int, block: int):
    """Two 32-bit keys (as signed ints) for one (tensor, block) stream."""
    h = _splitmix64(_splitmix64(seed & _M64) ^ (tensor_id << 40) ^ block)
    return _i32(h), _i32(h >> 32)


def _fmix32(x: torch.Tensor) -> torch.Tensor:
    """The 32-bit finaliser of MurmurHash3 on an int32 tensor (wrapping multiply; the logical
    right shifts are arithmetic shifts with the sign extension masked off)."""
    x = x ^ ((x >> 16) & 0xFFFF)
    x = x * _i32(0x85EBCA6B)
    x = x ^ ((x >> 13) & 0x7FFFF)
    x = x * _i32(0xC2B2AE35)
    return x ^ ((x >> 16) & 0xFFFF)


def normal_levels(seed: int, tensor_id: int, blocks, n: int, device) -> torch.Tensor:
    """f32 [len(blocks), n]: row i is the stream of (tensor_id, blocks[i]), n < 2**31 elements."""
    dev = torch.device(device)
    ka = torch.tensor([_keys(seed, tensor_id, b)[0] for b in blocks], dtype=torch.int32, device=dev)[:, None]
    kb = torch.tensor([_keys(seed, tensor_id, b)[1] for b in blocks], dtype=torch.int32, device=dev)[:, None]
    idx = torch.arange(n, dtype=torch.int32, device=dev)[None, :]
    h = _fmix32(_fmix32(idx ^ ka) + kb)
    level = ((h >> 16) & 0xFFFF).long()
    return _normal_table().to(dev)[level]


def outlier_channels(w: Workload) -> torch.Tensor:
    """int64 [Hkv, 4]: the channels of K scaled by 8, fixed per KV head."""
    g = _gen("cpu", w.seed ^ 0x0A11)
    return torch.stack([torch.randperm(HEAD_DIM, generator=g)[:4] for _ in range(w.n_kv_heads)])


def make_inputs(w: Workload, device="cpu", n_queries: int = 1, want_v_dense: bool = True, problems=None):
    """Draw one batch of inputs for workload `w` on `device` (bit-identical on every device).

    Returns a dict of tensors:
      k, v      bf16 [B, Hkv, T, 128]
      q         bf16 [n_queries, B, Hq, 128]   (independent query sets)
      scores    f32  [B, Hkv, T, S]
      tok_class u8   [B, T] or None            (None = every token routed)
      seq_len   i32  [B]
    With problems = [(b, hk), ...] only those (batch, kv head) problems are drawn, laid out as a
    batch of len(problems) sequences with one KV head each (k [n, 1, T, 128], q [n_queries, n, Gq, 128],
    tok_class [n, T], ...): exactly the slices of the full draw.
    """
    dev = torch.device(device)
    B, Hkv, Hq, T, S = w.batch, w.n_kv_heads, w.n_q_heads, w.t_cache, w.n_groups
    gq = w.gq
    out_ch = outlier_channels(w)
    scale_all = torch.ones(Hkv, 1, HEAD_DIM, dtype=torch.float32)
    for h in range(Hkv):
        scale_all[h, 0, out_ch[h]] = 8.0
    scale_all = scale_all.to(dev)
    if problems is None:
        groups = [[(b, h) for h in range(Hkv)] for b in range(B)]     # one sequence at a time
        nb, nh = B, Hkv
    else:
        groups = [[p] for p in problems]
        nb, nh = len(problems), 1
    k = torch.empty(nb, nh, T, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    v = torch.empty(nb, nh, T, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    scores = torch.empty(nb, nh, T, S, dtype=torch.float32, device=dev)
    for i, grp in enumerate(groups):          # per-group chunks bound the temporaries
        blocks = [b * Hkv + h for b, h in grp]
        heads = torch.tensor([h for _, h in grp], device=dev)
        kb = normal_levels(w.seed, _T_K, blocks, T * HEAD_DIM, dev).view(len(grp), T, HEAD_DIM)
        k[i] = (kb * scale_all[heads]).to(torch.bfloat16)
        del kb
        v[i] = normal_levels(w.seed, _T_V, blocks, T * HEAD_DIM, dev).view(len(grp), T, HEAD_DIM).to(torch.bfloat16)
        noise = normal_levels(w.seed, _T_SCORE, blocks, T * S, dev).view(len(grp), T, S)
        if w.score_recipe == "vnorm":
            # squares of bf16 values and their 128/S-term sums are exact in fp64, the square root is
            # correctly rounded: the same bits on every device
            vg = v[i].to(torch.float64).view(len(grp), T, S, HEAD_DIM // S)
            scores[i] = vg.pow(2).sum(-1).sqrt().to(torch.float32) + 0.5 * noise
        elif w.score_recipe == "normal":
            scores[i] = noise
        else:
            raise ValueError(w.score_recipe)
        del noise
    q_all = normal_levels(w.seed, _T_Q, list(range(n_queries)), B * Hq * HEAD_DIM, dev)
    q_all = q_all.view(n_queries, B, Hq, HEAD_DIM).to(torch.bfloat16)
    if problems is None:
        q = q_all
    else:
        q = torch.stack([q_all[:, b, h * gq:(h + 1) * gq] for b, h in problems], dim=1).contiguous()

    tok_class = None
    if w.n_text > 0:
        # Leading text tokens keep every group; the remaining tokens are the
        # survivors of the visual-token reducer and are routed.  The survivors'
        # contents are iid, so drawing T tokens directly equals gathering them
        # from the longer original sequence; the keep mask itself is still
        # drawn so the retained count is the recipe's, not an assumption.
        gc = _gen("cpu", w.seed ^ 0x7E57)
        n_keep = w.t_cache - w.n_text
        tok_class = torch.empty(B, T, dtype=torch.uint8)
        for b in range(B):
            keep = torch.randperm(w.n_visual_total, generator=gc)[:n_keep]
            assert keep.numel() == n_keep
            tok_class[b, : w.n_text] = CLS_FULL
            tok_class[b, w.n_text:] = CLS_ROUTED
        if problems is not None:
            tok_class = torch.stack([tok_class[b] for b, _ in problems])
        tok_class = tok_class.to(dev)
    seq_len = torch.full((nb,), T, dtype=torch.int32, device=dev)
    d = dict(k=k, v=v, q=q, scores=scores, tok_class=tok_class, seq_len=seq_len)
    if not want_v_dense:
        d.pop("v")
    return d


def problem_view(w: Workload, problems) -> Workload:
    """The workload `make_inputs(w, problems=...)` lays out: one sequence per listed problem."""
    return replace(w, batch=len(problems), n_q_heads=w.gq, n_kv_heads=1)


def shrink(w: Workload, **kw) -> Workload:
    """A smaller variant with the same structure, for parity tests."""
    return replace(w, **kw)
