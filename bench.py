"""Benchmark of the fused Slide Attention forward.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--variant auto]
    python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric

One step = one forward of the whole hot path (depthwise shift/deform convolution of K and V,
logits, softmax, aggregation) over one batch of seeded synthetic feature maps.  Prints ONE JSON
line (rank 0).  With N > 1 (torchrun) every rank runs the full batch on its own GPU: the batch
axis shards with no exchange, so there is no collective on the data path ("weak" scaling).

Timing: CUDA events on the launching stream around exactly K steps, barrier + synchronize on both
sides, max over ranks.  Inputs rotate over several buffer sets whose total size exceeds twice the
L2 capacity, so every step reads its inputs from HBM.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2304_04237_b200 import synth  # noqa: E402

METRIC = "slide_attn_fwd_query_pixels_per_s"
UNIT = "query-pixels/s"
FALLBACK_HBM_GBS = 6650.0
VARIANT_IDS = {"direct": 1, "mma": 2, "umma_ts": 5, "strip": 6, "tile": 8, "mma_wide": 9}


def algorithmic_bytes(cfg) -> int:
    """Minimal HBM traffic of one forward: q, k, v read once, out written once, fp32 weights
    of both convolutions and the bias read once."""
    n = cfg["B"] * cfg["H"] * cfg["W"]
    C = cfg["heads"] * cfg["head_dim"]
    k2 = cfg["ksize"] ** 2
    sz = 2 if cfg["dtype"] == "bf16" else 4
    return n * C * 4 * sz + 2 * C * k2 * k2 * 4 + (cfg["heads"] * k2 * 4 if cfg["has_bias"] else 0)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, bytes per launch) of the dominant kernel
# from one `ncu --set full` capture (profiles/).  It is tied to the kernel source by a hash: once
# the kernel changes, the figure no longer applies and `traffic` is reported as null.
NCU_TRAFFIC = {
    ("umma_ts", "c2"): {"bytes": 83.49e6,
                        "sources": ('paper_2304_04237_b200/csrc/umma_ts_kernel.cu', 'paper_2304_04237_b200/csrc/ptx.cuh'),
                        "sha256": "6c2f4e433aec8b8b57a0d6d1cc8f2be5a7dbd005c5f929bf5f1ac07841216743"},
    ("fixed_shift", "c2"): {"bytes": 85.38e6,
                            "sources": ('paper_2304_04237_b200/csrc/shift_kernel.cu', 'paper_2304_04237_b200/csrc/tile_common.cuh', 'paper_2304_04237_b200/csrc/ptx.cuh'),
                            "sha256": "d52af488501a9d58cb50407f1b82e038f60eae2056031d64999604761f99ad6c"},
}


def ncu_traffic(variant, workload):
    import hashlib
    rec = NCU_TRAFFIC.get((variant, workload))
    if rec is None:
        return None
    try:
        h = hashlib.sha256(b"".join(open(os.path.join(ROOT, f), "rb").read() for f in rec["sources"])).hexdigest()
    except OSError:
        return None
    return rec["bytes"] if h == rec["sha256"] else None


def other_rooflines(cfg, kernel_ms, fixed_shift=False):
    """The method's own arithmetic against the two compute ceilings, for context beside the HBM figure:
    2 C (2 k^4 + 2 k^2) flops per query pixel (2 C 2 k^2 with fixed-shift weights); fp32 ALU ceiling =
    SMs x 128 lanes x 2 x max SM clock; bf16 tensor ceiling = the measured cuBLAS figure (burst)."""
    k2 = cfg["ksize"] ** 2
    per_channel = 2 * k2 if fixed_shift else 2 * k2 * k2 + 2 * k2
    flops = 2.0 * cfg["heads"] * cfg["head_dim"] * per_channel * cfg["B"] * cfg["H"] * cfg["W"]
    out = {"flops_per_launch": flops}
    if not kernel_ms or kernel_ms <= 0:
        return out
    tf = flops / (kernel_ms * 1e-3) / 1e12
    out["achieved_tflops"] = tf
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            mp = json.load(f)
        alu = 148 * 128 * 2 * float(mp["sm_max_mhz"]) * 1e6 / 1e12
        out.update({"fp32_alu_peak_tflops": alu, "frac_fp32_alu_peak": tf / alu,
                    "bf16_tensor_peak_tflops": float(mp["bf16_tflops"]),
                    "frac_bf16_tensor_peak": tf / float(mp["bf16_tflops"])})
    except Exception:
        pass
    return out


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what a batch sharded over `world` ranks takes (no data-path collective;
    this all-reduce of one number is the only exchange)."""
    if world == 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, units_per_rank: int, ms_per_step: float) -> float:
    """Weak scaling: every rank processes its own full batch, so the job's rate is the sum."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": (float(np.median(self.samples)) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def cpu_oracle_rate(cfg, x, budget_s=15.0):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: whole images
    taken from the front of the batch, the pass repeated until about `budget_s` seconds of
    work are done.  Returns (pixels/s, threads, description)."""
    import oracle
    hw = cfg["H"] * cfg["W"]
    nb = min(2, x["q"].shape[0])
    args = lambda n: (x["q"][:n], x["k"][:n], x["v"][:n], x["wk"], x["wv"], x["bias"], cfg["ksize"])
    t0 = time.perf_counter()
    oracle.forward(*args(nb))
    per_img = (time.perf_counter() - t0) / nb
    n_img = int(max(1, min(x["q"].shape[0], budget_s / max(per_img, 1e-9))))
    reps = int(max(1, min(50, budget_s / max(per_img * n_img, 1e-9))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.forward(*args(n_img))
    dt = time.perf_counter() - t0
    return (reps * n_img * hw / dt, oracle.threads(),
            f"first {n_img} of {cfg['B']} images of the workload, {reps} passes "
            f"({reps * n_img * hw} query pixels, {dt:.1f} s)")


def kernel_only(sa, torch, name, variant_id, launches=300, warm_l2=False):
    """Dominant-kernel duration of another workload (a few hundred profiled forwards over rotating
    buffer sets; one resident set when `warm_l2`): for the roofline figures reported beside the
    headline workload's."""
    cfg = dict(synth.CONFIGS[name])
    x = synth.make_inputs(**cfg)
    td = torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32
    host = {n: torch.from_numpy(x[n]).to(td) for n in ("q", "k", "v")}
    wk, wv = torch.from_numpy(x["wk"]).cuda(), torch.from_numpy(x["wv"]).cuda()
    bias = None if x["bias"] is None else torch.from_numpy(x["bias"]).cuda()
    l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
    set_bytes = 4 * host["q"].numel() * host["q"].element_size()
    n_sets = 1 if warm_l2 else max(2, int(np.ceil(2.0 * l2 / set_bytes)) + 1)
    sets = []
    for _ in range(n_sets):
        d = {n: host[n].cuda() for n in ("q", "k", "v")}
        d["out"] = torch.empty_like(d["q"])
        sets.append(d)
    ctx = sa.slide_attn_create(cfg["B"], cfg["H"], cfg["W"], cfg["heads"], cfg["head_dim"], cfg["ksize"], td, cfg["has_bias"])
    try:
        if variant_id:
            sa.slide_attn_set_variant(ctx, variant_id)
        stream = torch.cuda.current_stream()
        for i in range(20):
            d = sets[i % n_sets]
            sa.slide_attn_forward(ctx, d["q"], d["k"], d["v"], wk, wv, bias, d["out"], stream)
        torch.cuda.synchronize()
        sa.slide_attn_profile_begin(ctx)
        for i in range(launches):
            d = sets[i % n_sets]
            sa.slide_attn_forward(ctx, d["q"], d["k"], d["v"], wk, wv, bias, d["out"], stream)
        torch.cuda.synchronize()
        fwd_ms, main_ms, n = sa.slide_attn_profile_end(ctx)
        assert sa.slide_attn_query_status(ctx) == sa.OK
    finally:
        sa.slide_attn_destroy(ctx)
    peak, _ = hbm_peak()
    ab = algorithmic_bytes(cfg)
    return {"kernel_ms": main_ms, "forward_ms": fwd_ms, "launches": n, "algorithmic_bytes_per_launch": ab,
            "achieved": ab / (main_ms * 1e-3) / 1e9, "frac": ab / (main_ms * 1e-3) / 1e9 / peak,
            "l2": "warm (one resident buffer set)" if warm_l2 else f"cold ({n_sets} rotating buffer sets)"}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores; rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = dict(synth.CONFIGS[args.workload])
    # inputs for as many images as one step's sample may need
    x = synth.make_inputs(batch_limit=min(cfg["B"], 16), **cfg)
    import oracle
    hw = cfg["H"] * cfg["W"]
    t0 = time.perf_counter()
    oracle.forward(x["q"][:1], x["k"][:1], x["v"][:1], x["wk"], x["wv"], x["bias"], cfg["ksize"])
    per_img = time.perf_counter() - t0
    total_steps = args.steps + args.warmup
    n_img = int(max(1, min(x["q"].shape[0], 60.0 / total_steps / max(per_img, 1e-9))))
    call = lambda: oracle.forward(x["q"][:n_img], x["k"][:n_img], x["v"][:n_img], x["wk"], x["wv"],
                                  x["bias"], cfg["ksize"])
    for _ in range(args.warmup):
        call()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        call()
    dt = time.perf_counter() - t0
    value = args.steps * n_img * hw / dt
    sample = f"each step = first {n_img} of {cfg['B']} images ({n_img * hw} query pixels)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(cfg, args.workload, None),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, name, l2_note):
    c = {"workload": f"{name}: B={cfg['B']} H={cfg['H']} W={cfg['W']} heads={cfg['heads']} "
                     f"head_dim={cfg['head_dim']} k={cfg['ksize']} {cfg['dtype']} "
                     f"bias={'yes' if cfg['has_bias'] else 'no'} sigma_w={cfg['sigma_w']}",
         "name": name, "B": cfg["B"], "H": cfg["H"], "W": cfg["W"], "heads": cfg["heads"],
         "head_dim": cfg["head_dim"], "ksize": cfg["ksize"], "storage_dtype": cfg["dtype"]}
    if l2_note:
        c["l2"] = l2_note
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--workload", default="c2", choices=sorted(synth.CONFIGS))
    ap.add_argument("--variant", default="auto", choices=["auto"] + sorted(VARIANT_IDS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other", action="store_true", help="skip the kernel-only figures of the other gated shapes")
    ap.add_argument("--backward", type=int, default=20, metavar="N",
                    help="also time N backward passes (slide_attn_backward) of the workload and report them beside the forward "
                         "(single-GPU runs, window sizes the backward supports; 0 = off)")
    ap.add_argument("--block", type=int, default=200, metavar="N",
                    help="also time N whole blocks (slide_attn_block_forward: Eq. 1 projections, attention, Eq. 3 projection) "
                         "on the workload's shape and report them beside the forward (single-GPU runs, bf16; 0 = off)")
    ap.add_argument("--fixed-shift", action="store_true",
                    help="the workload with exactly one-hot depthwise weights (sigma_w = 0), run in fixed-shift mode")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2304_04237_b200 as sa

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = dict(synth.CONFIGS[args.workload])
    if args.fixed_shift:
        cfg["sigma_w"] = 0.0
    x = synth.make_inputs(**cfg)
    td = torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32
    host = {n: torch.from_numpy(x[n]).to(td) for n in ("q", "k", "v")}
    wk, wv = torch.from_numpy(x["wk"]).cuda(), torch.from_numpy(x["wv"]).cuda()
    bias = None if x["bias"] is None else torch.from_numpy(x["bias"]).cuda()

    # rotating buffer sets: total > 2 x L2 so that no step finds its inputs in cache
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    set_bytes = 4 * host["q"].numel() * host["q"].element_size()
    n_sets = max(2, int(np.ceil(2.0 * l2 / set_bytes)) + 1)
    sets = []
    for i in range(n_sets):
        s = {n: host[n].cuda() for n in ("q", "k", "v")}
        s["out"] = torch.empty_like(s["q"])
        sets.append(s)
    l2_note = (f"{n_sets} rotating (q,k,v,out) buffer sets, {n_sets * set_bytes / 1e6:.0f} MB in total "
               f"> 2 x L2 ({l2 / 1e6:.0f} MB)")

    ctx = sa.slide_attn_create(cfg["B"], cfg["H"], cfg["W"], cfg["heads"], cfg["head_dim"],
                               cfg["ksize"], td, cfg["has_bias"])
    if args.variant != "auto":
        sa.slide_attn_set_variant(ctx, VARIANT_IDS[args.variant])
    variant = {v: k for k, v in VARIANT_IDS.items()}[sa.slide_attn_get_variant(ctx)]
    if args.fixed_shift:
        sa.slide_attn_set_fixed_shift(ctx, True)
        variant = "fixed_shift"
    launches = sa.slide_attn_launches_per_forward(ctx)
    stream = torch.cuda.current_stream()

    def step(i):
        s = sets[i % n_sets]
        sa.slide_attn_forward(ctx, s["q"], s["k"], s["v"], wk, wv, bias, s["out"], stream)

    def fence():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    fence()

    # Headline: exactly K steps, nothing but the forwards between the two events (no kernel-timing
    # events inside).  When K steps are short, the timed region is repeated so that the clock samples
    # and the spread mean something; the median repeat is the reported one, the minimum goes beside it.
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    repeat_ms = []
    t_begin = time.perf_counter()
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            step(i)
        e1.record(stream)
        fence()
        repeat_ms.append(e0.elapsed_time(e1) / args.steps)
        if len(repeat_ms) >= 50 or (time.perf_counter() - t_begin >= 0.25 and len(repeat_ms) >= 3):
            break
    clocks = sampler.stop()
    assert sa.slide_attn_query_status(ctx) == sa.OK
    ms_per_step = max_over_ranks(float(np.median(repeat_ms)), world, "cuda")
    npx = cfg["B"] * cfg["H"] * cfg["W"]
    value = whole_job_value(world, npx, ms_per_step)

    # Second pass with the library's kernel-timing events on: duration of the dominant kernel alone.
    def kernel_pass(n, stepper):
        sa.slide_attn_profile_begin(ctx)
        for i in range(n):
            stepper(i)
        fence()
        return sa.slide_attn_profile_end(ctx)

    fwd_ms, main_ms, n_prof = kernel_pass(min(max(args.steps, 200), 1000), step)
    assert sa.slide_attn_query_status(ctx) == sa.OK

    # optional: the backward pass of the same workload (gradients of all six inputs)
    backward = None
    if args.backward > 0 and world == 1 and cfg["ksize"] <= 3 and cfg["head_dim"] == 32:
        s0 = sets[0]
        g = torch.randn_like(s0["q"])
        dq, dk, dv = (torch.empty_like(s0["q"]) for _ in range(3))
        dwk, dwv = torch.empty_like(wk), torch.empty_like(wv)
        dbias = None if bias is None else torch.empty_like(bias)
        call = lambda d: sa.slide_attn_backward(ctx, d["q"], d["k"], d["v"], wk, wv, bias, g, dq, dk, dv, dwk, dwv, dbias, stream)
        for i in range(3):
            call(sets[i % n_sets])
        fence()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(args.backward):
            call(sets[i % n_sets])
        b.record(stream)
        fence()
        assert sa.slide_attn_query_status(ctx) == sa.OK
        bms = a.elapsed_time(b) / args.backward
        backward = {"ms_per_step": bms, "steps": args.backward, "value": npx / (bms * 1e-3), "unit": UNIT,
                    "kernels": "weight transpose, point kernel (a, dl, dq, dbias), gather kernel (dk, dv), weight kernel (dWk, dWv)"}

    # optional: a whole block on the workload's shape (projections on tcgen05 around the attention stage)
    block = None
    if args.block > 0 and world == 1 and cfg["dtype"] == "bf16":
        C = cfg["heads"] * cfg["head_dim"]
        gen = torch.Generator(device="cuda").manual_seed(1234)
        xs = [torch.randn((cfg["B"], cfg["H"], cfg["W"], C), device="cuda", generator=gen).to(torch.bfloat16) for _ in range(2)]
        w_qkv = torch.randn((3, C, C), device="cuda", generator=gen) / C ** 0.5
        w_o = torch.randn((C, C), device="cuda", generator=gen) / C ** 0.5
        bout = torch.empty_like(xs[0])
        ys = [torch.empty_like(xs[0]) for _ in range(3)]

        def timed(fn, n):
            for i in range(3):
                fn(i)
            fence()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n):
                fn(i)
            b.record(stream)
            fence()
            assert sa.slide_attn_query_status(ctx) == sa.OK
            return a.elapsed_time(b) / n

        blk_ms = timed(lambda i: sa.slide_attn_block_forward(ctx, xs[i & 1], w_qkv, w_o, wk, wv, bias, bout, stream), args.block)
        qkv_ms = timed(lambda i: sa.slide_attn_project(ctx, xs[i & 1], w_qkv, ys, stream), args.block)
        o_ms = timed(lambda i: sa.slide_attn_project(ctx, xs[i & 1], w_o, [bout], stream), args.block)
        tok_bytes = npx * C * 2
        block = {"ms_per_step": blk_ms, "steps": args.block, "value": npx / (blk_ms * 1e-3), "unit": UNIT,
                 "proj_qkv_ms": qkv_ms, "proj_qkv_gbs": 4 * tok_bytes / (qkv_ms * 1e-3) / 1e9,
                 "proj_o_ms": o_ms, "proj_o_gbs": 2 * tok_bytes / (o_ms * 1e-3) / 1e9,
                 "bytes_min_three_stages": 10 * tok_bytes, "bytes_min_fused": 2 * tok_bytes,
                 "kernels": "projection GEMM (Eq. 1, three outputs), attention (prep + main), projection GEMM (Eq. 3)"}

    # end to end through the host-buffer entry point: pinned host inputs in, pinned result out
    e2e = None
    if args.e2e_steps > 0:
        pin = {n: host[n].pin_memory() for n in ("q", "k", "v")}
        pwk, pwv = torch.from_numpy(x["wk"]).pin_memory(), torch.from_numpy(x["wv"]).pin_memory()
        pb = None if x["bias"] is None else torch.from_numpy(x["bias"]).pin_memory()
        pout = torch.empty_like(pin["q"]).pin_memory()
        for _ in range(2):
            sa.slide_attn_forward_host(ctx, pin["q"], pin["k"], pin["v"], pwk, pwv, pb, pout, stream)
        fence()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.e2e_steps):
            sa.slide_attn_forward_host(ctx, pin["q"], pin["k"], pin["v"], pwk, pwv, pb, pout, stream)
        b.record(stream)
        fence()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / args.e2e_steps, world, "cuda")
        h2d = 3 * pin["q"].numel() * pin["q"].element_size() + 2 * pwk.numel() * 4 + (0 if pb is None else pb.numel() * 4)
        e2e = {"value": whole_job_value(world, npx, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(pout.numel() * pout.element_size()),
               "steps": args.e2e_steps}
    sa.slide_attn_destroy(ctx)

    other = None
    if rank == 0 and world == 1 and not args.no_other and not args.fixed_shift:
        vid = 0 if args.variant == "auto" else VARIANT_IDS[args.variant]
        del sets
        torch.cuda.empty_cache()
        other = {}
        for name in ("c2", "c3", "c5"):
            if name != args.workload:
                other[name] = kernel_only(sa, torch, name, vid)
        other["c5_warm_l2"] = kernel_only(sa, torch, "c5", vid, warm_l2=True)

    if rank == 0:
        peak, peak_src = hbm_peak()
        abytes = algorithmic_bytes(cfg)
        achieved = abytes / (main_ms * 1e-3) / 1e9 if main_ms > 0 else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if cfg["dtype"] == "f32" else "bf16 storage, f32 accumulate",
            "data": "synthetic", "config": workload_config(cfg, args.workload, l2_note),
            "variant": variant, "gpu_launches": launches * args.steps,
            "hbm_gbs_algorithmic": abytes / (ms_per_step * 1e-3) / 1e9,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": (achieved / peak if achieved else None),
                         "traffic": ncu_traffic(variant, args.workload),
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": abytes,
                         "kernel_ms": main_ms, "forward_ms": fwd_ms, "launches_averaged": n_prof,
                         "other": other},
            "timing": {"repeats": len(repeat_ms), "steps_per_repeat": args.steps, "reported": "median repeat",
                       "median_ms_per_step": float(np.median(repeat_ms)), "min_ms_per_step": float(min(repeat_ms)),
                       "max_ms_per_step": float(max(repeat_ms))},
            "compute_ceilings": other_rooflines(cfg, main_ms, args.fixed_shift),
            "clocks": clocks, "e2e": e2e,
        }
        if backward:
            line["backward"] = backward
        if block:
            line["block"] = block
        if world == 1 and not args.no_cpu_baseline:
            v, cores, sample = cpu_oracle_rate(cfg, x)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
