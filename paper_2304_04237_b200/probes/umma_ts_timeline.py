"""Where the roles of umma_ts_kernel spend their time (CTA 0), from the time-line build of the library
(python -m paper_2304_04237_b200.build --timeline): mean and maximum cycles of every wait and of the work between the
waits, for one product warp (and its softmax), one value warp and the two MMA-issuing roles.

    python paper_2304_04237_b200/probes/umma_ts_timeline.py [workload]
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
    cfg = synth.CONFIGS[name]
    x = synth.make_inputs(**cfg)
    B, H, W, heads = cfg["B"], cfg["H"], cfg["W"], cfg["heads"]
    dev = {n: torch.from_numpy(x[n]).to(torch.bfloat16).cuda() for n in ("q", "k", "v")}
    dev.update({n: torch.from_numpy(x[n]).cuda() for n in ("wk", "wv", "bias")})
    out = torch.empty_like(dev["q"])
    ctx = sa.slide_attn_create(B, H, W, heads, 32, 3, torch.bfloat16, True)
    for _ in range(3):
        sa.slide_attn_forward(ctx, dev["q"], dev["k"], dev["v"], dev["wk"], dev["wv"], dev["bias"], out)
    torch.cuda.synchronize()
    assert sa.slide_attn_query_status(ctx) == sa.OK
    buf = (ctypes.c_longlong * (16 * 128))()
    assert binding.load().slide_attn_umma_ts_timeline(buf) == 0
    sa.slide_attn_destroy(ctx)
    t = np.array(buf).reshape(16, 128)
    n = int(np.count_nonzero(t[9]))                      # chunks the value warp consumed
    print(f"{name}: {n} chunks ({n / 3:.1f} blocks of 128 pixels) in CTA 0; cycles, first two blocks left out")

    def span(a, b):
        m = (t[a] != 0) & (t[b] != 0)
        m[:6] = False
        d = (t[b] - t[a])[m]
        return (int(d.mean()), int(d.max()), int(m.sum())) if m.any() else (0, 0, 0)

    rows = [("product warp: wait for a free P buffer", 0, 1), ("product warp: products, store, hand over", 1, 2),
            ("softmax: wait for the logits", 3, 4), ("softmax: weights of 32 pixels", 4, 5), ("softmax: wait for a free A' tile", 5, 6),
            ("value warp: wait for a chunk", 7, 8), ("value warp: one chunk (loads, widenings, FMAs)", 8, 9),
            ("key MMA thread: wait for P", 10, 11), ("key MMA thread: issue 6 MMAs + commit", 11, 12),
            ("value MMA thread: wait for a free slot", 13, 14), ("value MMA thread: issue 2 MMAs + commit", 14, 15)]
    print("| span | mean | max | samples |\n|---|---|---|---|")
    for label, a, b in rows:
        print("| %s | %d | %d | %d |" % ((label,) + span(a, b)))
    done = t[9][:n]
    per_block = (done[n - 1] - done[5]) / ((n - 6) / 3.0)
    print(f"value warp, cycles per block (last chunk to last chunk): {per_block:.0f}")


if __name__ == "__main__":
    main()
