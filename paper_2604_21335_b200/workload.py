"""Seeded synthetic inputs shaped like the paper's decode workloads.

This module only draws random tensors and lays them out; it contains none of
the method's arithmetic (no page bounds, no selection, no routing, no
attention), so both the CUDA path and the CPU checker can be fed from it.

Shapes follow the paper's settings: LLaMA-2-7B-like multi-head attention,
Qwen2.5-7B-like grouped-query attention, a LLaVA-1.5-7B-like cache of 576
visual + text tokens reduced to a quarter of the visual tokens (Appendix
"Training Details and Implementation Cost", VLM paragraph), value groups
S in {8, 16} with K/S budgets from Section 3.3 / Appendix C.

Value recipe (all configs): Q, K, V iid N(0,1) rounded to bf16; in K, four
channels per KV head (ids drawn once per head from the seed) are multiplied
by 8 before rounding.  Router scores are fp32 per (batch, kv head, token,
group): iid N(0,1), or the L2 norm of the bf16 value group plus N(0, 0.5).
"""
from __future__ import annotations

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


def outlier_channels(w: Workload) -> torch.Tensor:
    """int64 [Hkv, 4]: the channels of K scaled by 8, fixed per KV head."""
    g = _gen("cpu", w.seed ^ 0x0A11)
    return torch.stack([torch.randperm(HEAD_DIM, generator=g)[:4] for _ in range(w.n_kv_heads)])


def make_inputs(w: Workload, device="cpu", n_queries: int = 1, want_v_dense: bool = True):
    """Draw one batch of inputs for workload `w` on `device`.

    Returns a dict of tensors:
      k, v      bf16 [B, Hkv, T, 128]
      q         bf16 [n_queries, B, Hq, 128]   (independent query sets)
      scores    f32  [B, Hkv, T, S]
      tok_class u8   [B, T] or None            (None = every token routed)
      seq_len   i32  [B]
    """
    dev = torch.device(device)
    B, Hkv, Hq, T, S = w.batch, w.n_kv_heads, w.n_q_heads, w.t_cache, w.n_groups
    g = _gen(dev, w.seed)
    out_ch = outlier_channels(w).to(dev)

    k = torch.empty(B, Hkv, T, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    v = torch.empty(B, Hkv, T, HEAD_DIM, dtype=torch.bfloat16, device=dev)
    scores = torch.empty(B, Hkv, T, S, dtype=torch.float32, device=dev)
    scale = torch.ones(Hkv, 1, HEAD_DIM, dtype=torch.float32, device=dev)
    for h in range(Hkv):
        scale[h, 0, out_ch[h]] = 8.0
    for b in range(B):  # per-sequence chunks bound the fp32 temporaries
        kb = torch.randn(Hkv, T, HEAD_DIM, generator=g, device=dev, dtype=torch.float32)
        k[b] = (kb * scale).to(torch.bfloat16)
        del kb
        vb = torch.randn(Hkv, T, HEAD_DIM, generator=g, device=dev, dtype=torch.float32)
        v[b] = vb.to(torch.bfloat16)
        del vb
        noise = torch.randn(Hkv, T, S, generator=g, device=dev, dtype=torch.float32)
        if w.score_recipe == "vnorm":
            vg = v[b].to(torch.float32).view(Hkv, T, S, HEAD_DIM // S)
            scores[b] = vg.pow(2).sum(-1).sqrt() + 0.5 * noise
        elif w.score_recipe == "normal":
            scores[b] = noise
        else:
            raise ValueError(w.score_recipe)
    q = torch.randn(n_queries, B, Hq, HEAD_DIM, generator=g, device=dev,
                    dtype=torch.float32).to(torch.bfloat16)

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
        tok_class = tok_class.to(dev)
    seq_len = torch.full((B,), T, dtype=torch.int32, device=dev)
    d = dict(k=k, v=v, q=q, scores=scores, tok_class=tok_class, seq_len=seq_len)
    if not want_v_dense:
        d.pop("v")
    return d


def shrink(w: Workload, **kw) -> Workload:
    """A smaller variant with the same structure, for parity tests."""
    return replace(w, **kw)
