"""The benchmark's byte accounting and CPU reference arm, without a GPU: the algorithmic bytes of
a step follow from the shapes alone (they are what `value` and `roofline.achieved` divide by the
measured time), and the reference arm prints the contract's JSON line."""
import json
import subprocess
import sys
from pathlib import Path

import bench
from paper_2604_21335_b200 import workload as W

ROOT = Path(__file__).resolve().parent.parent


def test_algorithmic_bytes_of_the_llama_shaped_step():
    w = W.get("cfg1")                                   # 1 x 32 heads x 32768 tokens, S = 8, keep 4, budget 2048
    tok, pages = 32 * 32768, 32 * 2048
    sel_pages, sel_tokens = 32 * 128, 32 * 2048
    ab = bench.algorithmic_bytes(w, [32768], n_routed=tok, n_full=0, total_groups=tok * 4, sel_pages=sel_pages,
                                 sel_tokens=sel_tokens, sel_groups=sel_tokens * 4)
    assert ab["page_meta"] == tok * 256 + pages * 512 == 301989888
    assert ab["route_mask"] == tok * 8 * 4 + tok * 2
    assert ab["pack_values"] == tok * 4 * 32 * 2 + (tok + 32) * 4          # kept groups in and out, offsets
    assert ab["quest_select"] == pages * 512 + 32 * 256 + sel_pages * 4 + 32 * 4
    assert ab["decode_attn"] == sel_tokens * (256 + 2) + sel_tokens * 4 * 32 + sel_pages * 8 + 32 * (256 + 512)
    # stored value bytes really are K/S of the dense ones (Section 3.3, compression ratio)
    assert tok * 4 * 32 == tok * 256 // 2


def test_algorithmic_bytes_without_selection_and_with_classes():
    w = W.get("cfg3")                                   # Quest off, 128 full-width text tokens per sequence
    seq = [w.t_cache] * w.batch
    tok = sum(seq) * w.n_kv_heads
    n_full = 128 * w.batch * w.n_kv_heads
    ab = bench.algorithmic_bytes(w, seq, n_routed=tok - n_full, n_full=n_full,
                                 total_groups=(tok - n_full) * 3 + n_full * 8, sel_pages=17 * w.n_problems,
                                 sel_tokens=tok, sel_groups=(tok - n_full) * 3 + n_full * 8)
    assert ab["quest_select"] == 0
    assert ab["route_mask"] == (tok - n_full) * 8 * 4 + tok + tok * 2      # scores of routed tokens, classes, masks
    groups = (tok - n_full) * 3 + n_full * 8
    assert ab["decode_attn"] == tok * 258 + groups * 32 + 17 * w.n_problems * 8 + w.batch * w.n_q_heads * 768


def test_reference_arm_prints_the_contract_line():
    p = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "cfg0",
                        "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads([x for x in p.stdout.splitlines() if x.startswith("{")][-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert line["steps"] == 1 and line["n_gpus"] == 1 and line["higher_is_better"] is True
