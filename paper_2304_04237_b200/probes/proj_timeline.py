"""Time line of the projection kernel's role loops (CTA 0) on a workload's shape, from the time-line build of the
library (python -m paper_2304_04237_b200.build --timeline).  Prints, per work item, the clock64 stamps (cycles from the
first one): MMA thread turns to the item / its accumulator slot is free / MMAs and commit issued; the owning epilogue
group's first warp turns to the item / sees the accumulator / has stored it.

    python paper_2304_04237_b200/probes/proj_timeline.py [workload] [nmat]
"""
import ctypes
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
from paper_2304_04237_b200 import binding, synth  # noqa: E402

binding.LIB_PATH = os.path.join(HERE, "_build", "libslide_attn_timeline.so")
import paper_2304_04237_b200 as sa  # noqa: E402


def main():
    name = sys.argv[1] if len(sys.argv) > 1 else "c2"
    nmat = int(sys.argv[2]) if len(sys.argv) > 2 else 3
    cfg = synth.CONFIGS[name]
    B, H, W, heads, d = cfg["B"], cfg["H"], cfg["W"], cfg["heads"], cfg["head_dim"]
    C = heads * d
    ctx = sa.slide_attn_create(B, H, W, heads, d, 3, torch.bfloat16, False)
    x = torch.randn((B, H, W, C), device="cuda").to(torch.bfloat16)
    w = torch.randn((nmat, C, C), device="cuda") / C ** 0.5
    ys = [torch.empty_like(x) for _ in range(nmat)]
    for _ in range(3):
        sa.slide_attn_project(ctx, x, w, ys)
    torch.cuda.synchronize()
    assert sa.slide_attn_query_status(ctx) == sa.OK
    buf = (ctypes.c_longlong * (6 * 256))()
    assert binding.load().slide_attn_proj_timeline(buf) == 0
    sa.slide_attn_destroy(ctx)
    t = np.array(buf).reshape(6, 256)
    n = int(np.count_nonzero(t[2]))
    t0 = t[0][0]
    print(f"{name}: C = {C}, {nmat} output tensor(s), {n} work items in CTA 0 of the last launch")
    print("| item | MMA turns to it | slot free | commit issued | group turns to it | accumulator seen | stored |")
    print("|---|---|---|---|---|---|---|")
    for i in range(min(n, 24)):
        print("| %d | %d | %d | %d | %d | %d | %d |" % ((i,) + tuple(int(t[r][i] - t0) for r in range(6))))
    print(f"cycles per item (first to last MMA turn): {(t[0][n - 1] - t[0][0]) / max(1, n - 1):.0f}")


if __name__ == "__main__":
    main()
