#!/usr/bin/env python
"""Benchmark of the Stochastic Attention hot path on B200.

One step = one pass of the forward hot path over one batch of the Qwen3-8B-shaped
workload (bf16, B=1, 32 query / 8 KV heads, d=128, n=32768, w=1024): a fresh permutation
(sa_make_perm) followed by the gated SA+SWA forward (sa_swa_gated_forward), which runs the
fused SA kernel and then the plain SWA kernel, whose launch also applies the gates and
combines the two branches.  `value` is tokens/s of that step.
Beside it the JSON line reports the SA-only and SWA-only forward (tokens/s, TFLOP/s with
4*B*Hq*n*w*d nominal flops, SA overhead over SWA), the permutation alone, the backward on
the pre-training shape, a roofline entry for the SA forward kernel timed live with CUDA
events inside the step, an end-to-end number with host buffers, and the float64 CPU oracle
timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C3]
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SA fwd tokens/s (step = fresh permutation + gated SA+SWA forward)"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def event_ms(fn, iters, warmup, torch):
    """Mean milliseconds per call of fn, CUDA events on the current stream."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def oracle_sample_rate(c, t, rows_count, seed=0):
    """Times the float64 oracle (both branches + gate) on a random sample of query rows of
    workload c; returns (tokens/s extrapolated to whole tokens, seconds, rows, threads)."""
    import numpy as np

    import oracle
    from paper_2604_00754_b200.workloads import as_f64
    q, k, v = as_f64(t["q"]), as_f64(t["k"]), as_f64(t["v"])
    perm, inv = oracle.make_perm(c.seed, 0, c.B, c.n)
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(c.B * c.Hq * c.n, size=rows_count, replace=False)).astype(np.int64)
    lg = t["gate_logits"].double().numpy()
    t0 = time.perf_counter()
    ysa, _ = oracle.forward_rows(0, q, k, v, perm, inv, c.w, c.flags, rows)
    ysw, _ = oracle.forward_rows(1, q, k, v, None, None, c.w, c.flags, rows)
    g = 1 / (1 + np.exp(-lg))
    hq = (rows // c.n) % c.Hq
    y = g[0, hq][:, None] * ysa + g[1, hq][:, None] * ysw
    dt = time.perf_counter() - t0
    assert np.isfinite(y).all()
    tokens = rows_count / c.Hq          # a token is done when all its Hq rows are
    return tokens / dt, dt, rows_count, oracle.n_threads()


def run_reference(args, c):
    """Reference arm: the CPU oracle as it stands, on host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2604_00754_b200 import workloads as wl
    t = wl.draw(c)
    rows = 32768
    for _ in range(min(args.warmup, 1)):
        oracle_sample_rate(c, t, 1024)
    rates, secs = [], []
    for s in range(args.steps):
        r, dt, _, threads = oracle_sample_rate(c, t, rows, seed=s)
        rates.append(r)
        secs.append(dt)
    value = sum(rows / c.Hq for _ in rates) / sum(secs)
    sample = "%d random query rows (of %d) per step, both branches + gate, extrapolated" % (
        rows, c.B * c.Hq * c.n)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(c),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
    }))


def workload_config(c):
    return {"workload": c.name, "B": c.B, "Hq": c.Hq, "Hkv": c.Hkv, "n": c.n, "d": c.d, "w": c.w,
            "flags": "causal(original order)+circular window; SWA branch one-sided",
            "l2_policy": "inputs larger than L2 (Q+K+V+Y = %.0f MB per step)" % (
                2 * (2 * c.B * c.Hq + 2 * c.B * c.Hkv) * c.n * c.d / 1e6)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--n", type=int, default=0,
                    help="override the sequence length (profiling captures on a smaller case)")
    ap.add_argument("--leg", default="step",
                    choices=["step", "backward", "sa_fwd", "swa_fwd", "coverage", "gate"],
                    help="side measurements with their own JSON line (used for profiling): "
                         "backward = gated backward of the workload; sa_fwd / swa_fwd = that "
                         "branch's forward alone; coverage = the reach study of Prop. 2")
    ap.add_argument("--score-block", type=int, default=0, choices=[0, 64, 128],
                    help="force the score-block width of the tensor-core kernels (test hook of "
                         "the library; 0 = the library's own choice)")
    ap.add_argument("--gated-form", default="warps", choices=["warps", "epilogue"],
                    help="where the local branch's launch applies the gates: in its two idle warps "
                         "(scratch for the SA rows given: the default) or in the row threads' "
                         "epilogue (no scratch)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the side measurements (SWA, backward, e2e, CPU oracle)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2604_00754_b200 import workloads as wl
    c = {k.split("_")[0]: v for k, v in wl.CONFIGS.items()}[args.workload]
    if args.n:
        c = c.scaled(n=args.n, name="%s_n%d" % (c.name, args.n))
    if args.impl == "reference":
        run_reference(args, c)
        return

    import torch
    import torch.distributed as dist

    from paper_2604_00754_b200 import binding as sa
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sa.load_library()
    if args.score_block:
        sa.debug_set(sa.DEBUG_SCORE_BLOCK, args.score_block)
    pk = peaks()

    # Each rank holds its own batch of independent sequences (the path shards over
    # sequences and KV-head groups with no exchange step): weak scaling.
    cr = c.scaled(seed=c.seed + rank)
    host = wl.draw(cr, pin=True)
    dev = {k: v.cuda(non_blocking=True) for k, v in host.items()}
    q, k, v, lg = dev["q"], dev["k"], dev["v"], dev["gate_logits"]
    perm = torch.empty(c.B, c.n, dtype=torch.int32, device="cuda")
    inv = torch.empty_like(perm)
    y = torch.empty_like(q)
    prob = sa.SaProblem(B=c.B, n=c.n)
    ws = torch.empty(sa.sa_workspace_bytes(prob, sa.OP_MAKE_PERM), dtype=torch.uint8, device="cuda")
    out = {"y": y}
    # scratch for the SA branch's rows: the local branch's launch then combines with its idle warps
    gws = torch.empty(sa.sa_workspace_bytes(sa.make_problem(q, k, c.w, c.flags),
                                            sa.OP_GATED_FORWARD_SCRATCH),
                      dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()

    if args.leg == "backward":
        backward_leg(args, c, sa, torch, dev, perm, inv, ws, rank)
        return
    if args.leg in ("sa_fwd", "swa_fwd"):
        branch_leg(args, c, sa, torch, dev, perm, inv, ws, y, pk, rank)
        return
    if args.leg == "gate":
        gate_leg(args, c, sa, torch, pk, rank)
        return
    if args.leg == "coverage":
        if rank == 0:
            print(json.dumps({"leg": "coverage", "coverage_study": coverage_study(sa, torch, wl)}))
        return

    layer = [0]

    def step():
        sa.sa_make_perm(cr.seed, layer[0], c.B, c.n, perm=perm, inv=inv, ws=ws)
        sa.sa_swa_gated_forward(q, k, v, perm, inv, lg, c.w, c.flags, out=out,
                                ws=gws if args.gated_form == "warps" else None)
        layer[0] += 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    # timed region: K steps, the SA kernel of every step bracketed by its own event pair
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(args.steps)]
    for a, b in pairs:
        a.record(); b.record()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)
    launches0 = sa.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for a, b in pairs:
        sa.set_profile_events(a, b)
        step()
    e1.record()
    barrier()
    sa.set_profile_events(None, None)
    launches = sa.launch_count() - launches0
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    sa_kernel_ms = statistics.mean(a.elapsed_time(b) for a, b in pairs)
    if world > 1:
        tt = torch.tensor([total_ms], device="cuda")
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    assert sa.sa_read_status() == 0
    ms_per_step = total_ms / args.steps
    tokens_per_step = c.B * c.n * world
    value = tokens_per_step / (ms_per_step * 1e-3)

    flops_branch = 4.0 * c.B * c.Hq * c.n * c.w * c.d
    achieved = flops_branch / (sa_kernel_ms * 1e-3) / 1e12
    # DRAM bytes of one SA-branch launch: dram__bytes_read.sum + dram__bytes_write.sum of one ncu
    # capture of this kernel on this shape at n = 8192 (100.9 MB + 26.5 MB; the counter summary
    # is under profiles/), scaled by n because every tensor grows in proportion to it.
    traffic = None
    if (c.B, c.Hq, c.Hkv, c.d, c.w) == (1, 32, 8, 128, 1024):
        traffic = 127443200.0 * c.n / 8192
    sustained = args.steps * ms_per_step > 1500.0
    peak = pk["bf16_tflops_sustained"] if sustained else pk["bf16_tflops"]
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": workload_config(c), "clocks": clocks,
        "gpu_launches": int(launches),
        "roofline": {"kernel": "fused SA forward (gather, QK^T, softmax, PV, scatter); the gates are applied "
                               + ("by two idle warps of the local branch's launch"
                                  if args.gated_form == "warps"
                                  else "in the epilogue of the local branch's launch"),
                     "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak,
                     "peak_kind": "%s bf16 %s" % (pk["source"], "sustained" if sustained else "burst"),
                     "kernel_ms": sa_kernel_ms, "flops_per_launch": flops_branch,
                     "traffic": traffic,
                     "traffic_note": "ncu DRAM read+write of one launch at n=8192, scaled by n"},
    }

    if rank == 0 and not args.no_extras:
        line.update(extras(args, c, wl, sa, torch, dev, host, perm, inv, ws, y, pk))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def backward_leg(args, c, sa, torch, dev, perm, inv, ws, rank):
    """Gated forward once (saving what the backward needs), then `steps` timed backward passes."""
    q, k, v, lg = dev["q"], dev["k"], dev["v"], dev["gate_logits"]
    dy = torch.randn(q.shape, generator=torch.Generator(device="cuda").manual_seed(c.seed + 77),
                     device="cuda", dtype=torch.float32).to(q.dtype)
    sa.sa_make_perm(c.seed, 0, c.B, c.n, perm=perm, inv=inv, ws=ws)
    _, y_sa, y_swa, lse_sa, lse_swa = sa.sa_swa_gated_forward(q, k, v, perm, inv, lg, c.w, c.flags,
                                                              save_for_bwd=True)
    bws = torch.empty(sa.sa_workspace_bytes(sa.make_problem(q, k, c.w, c.flags), sa.OP_BACKWARD),
                      dtype=torch.uint8, device="cuda")
    out = {}

    def bwd():
        r = sa.sa_backward(q, k, v, perm, inv, lg, y_sa, y_swa, lse_sa, lse_swa, dy, c.w, c.flags,
                           ws=bws, out=out)
        out.update(zip(("dq", "dk", "dv", "dgate"), r))
    ms = event_ms(bwd, args.steps, args.warmup, torch)
    assert sa.sa_read_status() == 0
    flops = 2 * 2.5 * 4.0 * c.B * c.Hq * c.n * c.w * c.d
    if rank == 0:
        print(json.dumps({"leg": "backward", "metric": "gated SA+SWA backward tokens/s",
                          "value": c.B * c.n / (ms * 1e-3), "unit": "tokens/s", "ms_per_step": ms,
                          "steps": args.steps, "warmup": args.warmup,
                          "tflops_nominal": flops / (ms * 1e-3) / 1e12,
                          "config": workload_config(c), "dtype": "bf16", "data": "synthetic"}))


def branch_leg(args, c, sa, torch, dev, perm, inv, ws, y, pk, rank):
    """One branch's forward alone (the kernel the roofline entry is about, or its SWA twin)."""
    q, k, v = dev["q"], dev["k"], dev["v"]
    sa.sa_make_perm(c.seed, 0, c.B, c.n, perm=perm, inv=inv, ws=ws)
    if args.leg == "sa_fwd":
        fn = lambda: sa.sa_forward(q, k, v, perm, inv, c.w, c.flags, y=y)
    else:
        fn = lambda: sa.sa_swa_forward(q, k, v, c.w, c.flags, y=y)
    ms = event_ms(fn, args.steps, args.warmup, torch)
    assert sa.sa_read_status() == 0
    tf = 4.0 * c.B * c.Hq * c.n * c.w * c.d / (ms * 1e-3) / 1e12
    if rank == 0:
        print(json.dumps({"leg": args.leg, "ms": ms, "tokens_per_s": c.B * c.n / (ms * 1e-3),
                          "tflops_nominal": tf, "frac_of_burst": tf / pk["bf16_tflops"],
                          "steps": args.steps, "warmup": args.warmup,
                          "config": workload_config(c), "dtype": "bf16", "data": "synthetic"}))


def gate_leg(args, c, sa, torch, pk, rank):
    """Projection gates of Eq. 5-6 at the workload's model width (Hq*d) over B*n rows: dual-path
    forward and backward (what the counter summaries of those kernels are taken on)."""
    dm, rows = c.Hq * c.d, c.B * c.n
    gg = torch.Generator(device="cuda").manual_seed(17)
    ya = torch.randn(rows, dm, generator=gg, device="cuda").bfloat16()
    yb = torch.randn(rows, dm, generator=gg, device="cuda").bfloat16()
    wa = (torch.randn(dm, dm, generator=gg, device="cuda") * dm ** -0.5).bfloat16()
    wb = (torch.randn(dm, dm, generator=gg, device="cuda") * dm ** -0.5).bfloat16()
    og = torch.empty_like(ya)
    gbw = torch.empty(rows * dm * 8, dtype=torch.uint8, device="cuda")
    f_ms = event_ms(lambda: sa.sa_gate_projection_forward(ya, wa, yb, wb, out=og), args.steps,
                    args.warmup, torch)
    b_ms = event_ms(lambda: sa.sa_gate_projection_backward(og, ya, wa, yb, wb, ws=gbw), args.steps,
                    args.warmup, torch)
    gfl = 2.0 * rows * dm * dm
    if rank == 0:
        print(json.dumps({"leg": "gate", "rows": rows, "dm": dm, "fwd_dual_ms": f_ms,
                          "fwd_dual_tflops": 2 * gfl / (f_ms * 1e-3) / 1e12,
                          "bwd_dual_ms": b_ms, "bwd_dual_tflops": 6 * gfl / (b_ms * 1e-3) / 1e12,
                          "frac_of_burst_fwd": 2 * gfl / (f_ms * 1e-3) / 1e12 / pk["bf16_tflops"],
                          "frac_of_burst_bwd": 6 * gfl / (b_ms * 1e-3) / 1e12 / pk["bf16_tflops"]}))


def coverage_study(sa, torch, wl):
    """Fig. 2 (left) / Prop. 2 as numbers: seed-averaged |R_l| through sa_coverage for SA with an
    independent permutation per layer (the paper's default), SA with one fixed permutation reused
    at every layer (Sec. 3.3 deterministic mode), and plain SWA, beside Prop. 2's expansion
    bound applied to the measured mean; at the paper's n = 2048, w = 32 and at the (n, w) of the
    pre-training and the two Qwen3-shaped workloads.  Non-causal mask, as in the proposition."""
    import numpy as np
    out = {}
    cases = [("fig2_n2048_w32", 2048, 32, 6, 16), ("C5_n4096_w128", 4096, 128, 4, 8),
             ("C3_n32768_w1024", 32768, 1024, 3, 4), ("C4_n131072_w2048", 131072, 2048, 3, 2)]
    for name, n, w, L, seeds in cases:
        h = (w + 1) // 2 - 1
        band = min(n, 2 * h + 1)
        pr = (band - 1) / (n - 1)
        src = n // 3
        indep = np.zeros((seeds, L))
        fixed = np.zeros((seeds, L))
        t0 = time.perf_counter()
        for s_ in range(seeds):
            pl = [sa.sa_make_perm(9000 + s_, l, 1, n) for l in range(L)]
            perm = torch.cat([a for a, _ in pl]).contiguous()
            inv = torch.cat([b for _, b in pl]).contiguous()
            indep[s_] = sa.sa_coverage(perm, inv, w, 0, src, want_row_count=False)[2].cpu().numpy()
            p1 = pl[0][0].repeat(L, 1).contiguous()
            i1 = pl[0][1].repeat(L, 1).contiguous()
            fixed[s_] = sa.sa_coverage(p1, i1, w, 0, src, want_row_count=False)[2].cpu().numpy()
        ident = torch.arange(n, dtype=torch.int32, device="cuda").repeat(L, 1).contiguous()
        swa = sa.sa_coverage(ident, ident, w, 0, src, want_row_count=False)[2].cpu().numpy()
        torch.cuda.synchronize()
        mean = indep.mean(axis=0)
        bound = [float(band)] + [float((r + (n - r) * (1 - (1 - pr) ** r)).mean())
                                 for r in indep[:, :-1].T]
        out[name] = {"n": n, "w": w, "band": band, "layers": L, "seeds": seeds,
                     "sa_independent_sigma_mean_reach": [float(x) for x in mean],
                     "prop2_lower_bound_on_mean": bound,
                     "sa_fixed_sigma_mean_reach": [float(x) for x in fixed.mean(axis=0)],
                     "swa_reach": [int(x) for x in swa],
                     "swa_closed_form": [min(n, 2 * (l + 1) * h + 1) for l in range(L)],
                     "seconds": time.perf_counter() - t0}
    return out


def extras(args, c, wl, sa, torch, dev, host, perm, inv, ws, y, pk):
    """Side measurements on rank 0, outside the timed region of `value`."""
    q, k, v, lg = dev["q"], dev["k"], dev["v"], dev["gate_logits"]
    flops = 4.0 * c.B * c.Hq * c.n * c.w * c.d
    it = max(5, args.steps // 2)
    res = {}
    sa_ms = event_ms(lambda: sa.sa_forward(q, k, v, perm, inv, c.w, c.flags, y=y), it, 3, torch)
    swa_ms = event_ms(lambda: sa.sa_swa_forward(q, k, v, c.w, c.flags, y=y), it, 3, torch)
    perm_ms = event_ms(lambda: sa.sa_make_perm(c.seed, 1, c.B, c.n, perm=perm, inv=inv, ws=ws),
                       it, 3, torch)

    def side(ms):
        tf = flops / (ms * 1e-3) / 1e12
        return {"ms": ms, "tokens_per_s": c.B * c.n / (ms * 1e-3), "tflops": tf,
                "frac_of_burst": tf / pk["bf16_tflops"],
                "frac_of_sustained": tf / pk["bf16_tflops_sustained"],
                "frac_of_datasheet": tf / 2250.0}
    res["sa_fwd"] = side(sa_ms)
    res["swa_fwd"] = side(swa_ms)
    res["sa_overhead_vs_swa"] = sa_ms / swa_ms - 1.0
    res["make_perm_ms"] = perm_ms

    # end to end through the C entry point that takes HOST buffers: pinned host inputs ->
    # device, fresh permutation, gated forward, result back to pinned host memory, all inside
    # the timed region; the library pipelines the KV-head groups on three streams so that
    # copies in, kernels and copies out overlap
    hy = torch.empty_like(host["q"]).pin_memory()
    hg = host["gate_logits"].pin_memory()
    hws = torch.empty(sa.host_forward_ws_bytes(c.B, c.Hq, c.Hkv, c.n, c.d), dtype=torch.uint8,
                      device="cuda")
    layer = [1000]

    def e2e_step():
        sa.sa_swa_gated_forward_host(host["q"], host["k"], host["v"], hg, hy, c.w, c.flags,
                                     c.seed, layer[0], hws, n_groups=8, q_parts=2)
        layer[0] += 1
    e2e_ms = event_ms(e2e_step, it, 3, torch)
    elt = host["q"].element_size()
    res["e2e"] = {"value": c.B * c.n / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                  "h2d_bytes_per_step": sum(host[x].numel() for x in ("q", "k", "v")) * elt
                                        + hg.numel() * 4,
                  "d2h_bytes_per_step": hy.numel() * elt,
                  "api": "sa_swa_gated_forward_host (C ABI, host pointers), 8 KV-head groups, the "
                         "first and last cut in 2 query-head parts, on 3 streams"}
    del hws
    torch.cuda.empty_cache()

    # gated backward at the same workload (forward once, saving what the backward needs)
    if c.n * c.Hq <= 32768 * 32:
        dyb = torch.randn(q.shape, generator=torch.Generator(device="cuda").manual_seed(c.seed + 77),
                          device="cuda", dtype=torch.float32).to(q.dtype)
        sv = sa.sa_swa_gated_forward(q, k, v, perm, inv, lg, c.w, c.flags, save_for_bwd=True)
        bws3 = torch.empty(sa.sa_workspace_bytes(sa.make_problem(q, k, c.w, c.flags), sa.OP_BACKWARD),
                           dtype=torch.uint8, device="cuda")
        bo = {}

        def bwd_main():
            r = sa.sa_backward(q, k, v, perm, inv, lg, sv[1], sv[2], sv[3], sv[4], dyb, c.w,
                               c.flags, ws=bws3, out=bo)
            bo.update(zip(("dq", "dk", "dv", "dgate"), r))
        bms = event_ms(bwd_main, max(3, it // 2), 3, torch)
        bfl = 2 * 2.5 * flops
        res["backward_%s" % c.name.split("_")[0]] = {
            "gated_bwd_ms": bms, "tokens_per_s": c.B * c.n / (bms * 1e-3),
            "tflops_nominal": bfl / (bms * 1e-3) / 1e12,
            "frac_of_burst": bfl / (bms * 1e-3) / 1e12 / pk["bf16_tflops"]}
        del dyb, sv, bws3, bo
        torch.cuda.empty_cache()

    # rotary position embedding with original positions (Sec. 4.2): rotation inside the gather
    # of the SA forward against a rotation pass over Q and K followed by the plain forward
    cs, sn = sa.sa_rope_table(c.n, c.d, 1e6)
    qr, kr = torch.empty_like(q), torch.empty_like(k)
    fused_ms = event_ms(lambda: sa.sa_forward_rope(q, k, v, perm, inv, cs, sn, c.w, c.flags, y=y),
                        it, 3, torch)

    def unfused():
        sa.sa_rope_apply(q, k, cs, sn, out=qr)
        sa.sa_rope_apply(k, q, cs, sn, out=kr, kv=True)
        sa.sa_forward(qr, kr, v, perm, inv, c.w, c.flags, y=y)
    unfused_ms = event_ms(unfused, it, 3, torch)
    pass_ms = event_ms(lambda: (sa.sa_rope_apply(q, k, cs, sn, out=qr),
                                sa.sa_rope_apply(k, q, cs, sn, out=kr, kv=True)), it, 3, torch)
    res["rope"] = {"sa_fwd_rope_in_gather_ms": fused_ms, "rope_pass_plus_sa_fwd_ms": unfused_ms,
                   "rope_pass_ms": pass_ms, "sa_fwd_ms": sa_ms,
                   "pass_bytes": 2.0 * 2 * (q.numel() + k.numel()),
                   "pass_gbs": 2.0 * 2 * (q.numel() + k.numel()) / (pass_ms * 1e-3) / 1e9}
    del qr, kr, cs, sn
    torch.cuda.empty_cache()

    # single-layer SA forward on the HBM-bound shape: tokens/s and the achieved bytes per second
    # over the algorithmic bytes (Q, K, V in, Y out, each once)
    c2 = wl.C2
    t2 = {k_: v_.cuda() for k_, v_ in wl.draw(c2).items()}
    p2, i2 = sa.sa_make_perm(c2.seed, 0, c2.B, c2.n)
    # rotate among enough copies of the inputs to exceed L2 (134 MB per copy, L2 126 MB)
    copies = [{k_: t2[k_].clone() for k_ in ("q", "k", "v")} for _ in range(3)]
    y2 = torch.empty_like(t2["q"])
    turn = [0]

    def fwd2():
        cp = copies[turn[0] % len(copies)]
        turn[0] += 1
        sa.sa_forward(cp["q"], cp["k"], cp["v"], p2, i2, c2.w, c2.flags, y=y2)
    ms2 = event_ms(fwd2, max(20, it), 3, torch)
    bytes2 = 2.0 * (2 * c2.B * c2.Hq + 2 * c2.B * c2.Hkv) * c2.n * c2.d
    fl2 = 4.0 * c2.B * c2.Hq * c2.n * c2.w * c2.d
    res["C2_layer"] = {
        "sa_fwd_ms": ms2, "tokens_per_s": c2.B * c2.n / (ms2 * 1e-3),
        "algorithmic_bytes": bytes2, "achieved_gbs": bytes2 / (ms2 * 1e-3) / 1e9,
        "frac_of_hbm": bytes2 / (ms2 * 1e-3) / 1e9 / pk["hbm_gbs"],
        "tflops_nominal": fl2 / (ms2 * 1e-3) / 1e12,
        "l2_policy": "3 input copies in rotation (402 MB > L2)"}
    del t2, copies, y2
    torch.cuda.empty_cache()

    # long-context prefill: 48 layers back to back, each a fresh permutation + gated forward
    c4 = wl.C4
    t4 = {k_: v_.cuda() for k_, v_ in wl.draw(c4).items()}
    p4 = torch.empty(c4.B, c4.n, dtype=torch.int32, device="cuda")
    i4 = torch.empty_like(p4)
    y4 = torch.empty_like(t4["q"])
    ws4 = torch.empty(sa.sa_workspace_bytes(sa.SaProblem(B=c4.B, n=c4.n), sa.OP_MAKE_PERM),
                      dtype=torch.uint8, device="cuda")
    g4 = torch.empty(sa.sa_workspace_bytes(sa.make_problem(t4["q"], t4["k"], c4.w, c4.flags),
                                           sa.OP_GATED_FORWARD_SCRATCH), dtype=torch.uint8,
                     device="cuda")

    def prefill():
        for l in range(c4.layers):
            sa.sa_make_perm(c4.seed, l, c4.B, c4.n, perm=p4, inv=i4, ws=ws4)
            sa.sa_swa_gated_forward(t4["q"], t4["k"], t4["v"], p4, i4, t4["gate_logits"], c4.w,
                                    c4.flags, out={"y": y4}, ws=g4)
    ms4 = event_ms(prefill, 2, 3, torch)
    fl4 = 2 * 4.0 * c4.B * c4.Hq * c4.n * c4.w * c4.d * c4.layers
    res["C4_prefill_48_layers"] = {
        "total_ms": ms4, "ms_per_layer": ms4 / c4.layers,
        "tokens_per_s": c4.B * c4.n / (ms4 * 1e-3),
        "layer_tokens_per_s": c4.B * c4.n * c4.layers / (ms4 * 1e-3),
        "tflops_nominal": fl4 / (ms4 * 1e-3) / 1e12,
        "frac_of_sustained": fl4 / (ms4 * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
        "frac_of_burst": fl4 / (ms4 * 1e-3) / 1e12 / pk["bf16_tflops"]}
    del t4, p4, i4, y4, ws4, g4
    torch.cuda.empty_cache()

    # backward on the pre-training shape (fresh permutation, gated forward saving, backward)
    c5 = wl.C5
    t5 = {k_: v_.cuda() for k_, v_ in wl.draw(c5).items()}
    p5, i5 = sa.sa_make_perm(c5.seed, 0, c5.B, c5.n)
    saved = {}
    bout = {}
    bws = torch.empty(sa.sa_workspace_bytes(sa.make_problem(t5["q"], t5["k"], c5.w, c5.flags),
                                            sa.OP_BACKWARD), dtype=torch.uint8, device="cuda")

    def fwd5():
        r = sa.sa_swa_gated_forward(t5["q"], t5["k"], t5["v"], p5, i5, t5["gate_logits"], c5.w,
                                    c5.flags, save_for_bwd=True, out=saved)
        saved.update(zip(("y", "y_sa", "y_swa", "lse_sa", "lse_swa"), r))

    def bwd5():
        r = sa.sa_backward(t5["q"], t5["k"], t5["v"], p5, i5, t5["gate_logits"], saved["y_sa"],
                           saved["y_swa"], saved["lse_sa"], saved["lse_swa"], t5["dy"], c5.w,
                           c5.flags, ws=bws, out=bout)
        bout.update(zip(("dq", "dk", "dv", "dgate"), r))
    f5 = event_ms(fwd5, it, 3, torch)
    b5 = event_ms(bwd5, it, 3, torch)
    fl5 = 2 * 4.0 * c5.B * c5.Hq * c5.n * c5.w * c5.d
    ws5 = torch.empty(sa.sa_workspace_bytes(sa.SaProblem(B=c5.B, n=c5.n), sa.OP_MAKE_PERM),
                      dtype=torch.uint8, device="cuda")

    def step5():          # the pre-training step: 12 layers, a fresh permutation each
        for l in range(c5.layers):
            sa.sa_make_perm(c5.seed, l, c5.B, c5.n, perm=p5, inv=i5, ws=ws5)
            fwd5()
            bwd5()
    s5 = event_ms(step5, 3, 3, torch)
    bytes5 = 15 * 2.0 * c5.B * c5.Hq * c5.n * c5.d          # 15 tensor passes of 50.3 MB per layer
    res["pretrain_layer_C5"] = {
        "gated_fwd_ms": f5, "bwd_ms": b5, "tokens_per_s_fwd_bwd": c5.B * c5.n / ((f5 + b5) * 1e-3),
        "tflops_fwd_bwd": 3.5 * fl5 / ((f5 + b5) * 1e-3) / 1e12,
        "step_12_layers_ms": s5, "step_tokens_per_s": c5.B * c5.n / (s5 * 1e-3),
        "step_tflops_nominal": 3.5 * fl5 * c5.layers / (s5 * 1e-3) / 1e12,
        "hbm_floor_ms_per_layer": bytes5 / pk["hbm_gbs"] / 1e6,
        "frac_of_hbm_floor": (bytes5 / pk["hbm_gbs"] / 1e6) / (s5 / c5.layers)}
    del ws5
    del t5, saved, bout, bws
    torch.cuda.empty_cache()

    # the shape of the paper's efficiency table (Sec. 4.3, Table 3: B=16, H=16, d_h=64, w=256,
    # forward + backward of single-path SA); the paper's A100 / FlexAttention times are context
    t3 = {}
    paper_ms = {2048: 5.4, 4096: 7.9, 8192: 15.2, 16384: 29.6, 32768: 52.8}
    paper_full_ms = {2048: 8.0, 4096: 27.2, 8192: 99.7, 16384: 379.9, 32768: 1477.0}
    for n3 in (2048, 8192, 32768):
        c3 = wl.Workload("table3", "bf16", 16, 16, 16, n3, 64, 256, seed=9, ops="gated_fwd_bwd")
        d3 = {k_: v_.cuda() for k_, v_ in wl.draw(c3).items()}
        p3, i3 = sa.sa_make_perm(9, 0, c3.B, c3.n)
        y3 = torch.empty_like(d3["q"])
        l3 = torch.empty(c3.B, c3.Hq, c3.n, dtype=torch.float32, device="cuda")
        w3 = torch.empty(sa.sa_workspace_bytes(sa.make_problem(d3["q"], d3["k"], c3.w, c3.flags),
                                               sa.OP_BACKWARD), dtype=torch.uint8, device="cuda")
        o3 = {}

        def fb3():
            sa.sa_forward(d3["q"], d3["k"], d3["v"], p3, i3, c3.w, c3.flags, y=y3, lse=l3)
            r = sa.sa_backward(d3["q"], d3["k"], d3["v"], p3, i3, None, y3, None, l3, None,
                               d3["dy"], c3.w, c3.flags, ws=w3, out=o3)
            o3.update(zip(("dq", "dk", "dv", "dgate"), r))
        t3[str(n3)] = {"sa_fwd_bwd_ms": event_ms(fb3, 3, 3, torch),
                       "paper_a100_flexattention_ms": paper_ms[n3]}
        # the table's other column: full causal attention, here the same kernels with the
        # identity permutation and a window that covers the whole sequence
        ident = torch.arange(c3.n, dtype=torch.int32, device="cuda").repeat(c3.B, 1).contiguous()
        wfull = 2 * c3.n + 1

        def full3():
            sa.sa_forward(d3["q"], d3["k"], d3["v"], ident, ident, wfull, sa.CAUSAL, y=y3, lse=l3)
            r = sa.sa_backward(d3["q"], d3["k"], d3["v"], ident, ident, None, y3, None, l3, None,
                               d3["dy"], wfull, sa.CAUSAL, ws=w3, out=o3)
            o3.update(zip(("dq", "dk", "dv", "dgate"), r))
        t3[str(n3)]["full_attention_fwd_bwd_ms"] = event_ms(full3, 2, 3, torch)
        t3[str(n3)]["paper_a100_full_attention_ms"] = paper_full_ms[n3]
        del d3, y3, l3, w3, o3
        torch.cuda.empty_cache()
    res["table3_shape_B16_H16_d64_w256"] = t3

    # projection gates of Eq. 5-6 at the workload's model width (Hq*d), all B*n tokens: two
    # [B*n, dm] x [dm, dm] products on the tensor cores with the logistic and the combination
    # of the two paths in the epilogue; random bf16 Y and W stand in for attention outputs
    dm, rows_g = c.Hq * c.d, c.B * c.n
    gg = torch.Generator(device="cuda").manual_seed(17)
    ya = torch.randn(rows_g, dm, generator=gg, device="cuda").bfloat16()
    yb = torch.randn(rows_g, dm, generator=gg, device="cuda").bfloat16()
    wa = (torch.randn(dm, dm, generator=gg, device="cuda") * dm ** -0.5).bfloat16()
    wb = (torch.randn(dm, dm, generator=gg, device="cuda") * dm ** -0.5).bfloat16()
    og = torch.empty_like(ya)
    g2 = event_ms(lambda: sa.sa_gate_projection_forward(ya, wa, yb, wb, out=og), it, 3, torch)
    g1 = event_ms(lambda: sa.sa_gate_projection_forward(ya, wa, out=og), it, 3, torch)
    gfl = 2.0 * rows_g * dm * dm
    res["gate_projection"] = {
        "rows": rows_g, "dm": dm,
        "dual_ms": g2, "dual_tflops": 2 * gfl / (g2 * 1e-3) / 1e12,
        "dual_frac_of_burst": 2 * gfl / (g2 * 1e-3) / 1e12 / pk["bf16_tflops"],
        "single_ms": g1, "single_tflops": gfl / (g1 * 1e-3) / 1e12,
        "single_frac_of_burst": gfl / (g1 * 1e-3) / 1e12 / pk["bf16_tflops"]}
    # and their backward (dz, dy, dw: three products per path)
    gbw = torch.empty(rows_g * dm * 8, dtype=torch.uint8, device="cuda")
    gb2 = event_ms(lambda: sa.sa_gate_projection_backward(og, ya, wa, yb, wb, ws=gbw), 3, 3, torch)
    res["gate_projection"].update({
        "bwd_dual_ms": gb2, "bwd_dual_tflops": 6 * gfl / (gb2 * 1e-3) / 1e12,
        "bwd_dual_frac_of_burst": 6 * gfl / (gb2 * 1e-3) / 1e12 / pk["bf16_tflops"]})
    del ya, yb, wa, wb, og, gbw
    torch.cuda.empty_cache()

    res["coverage_study"] = coverage_study(sa, torch, wl)

    rate, dt, rows, threads = oracle_sample_rate(c, host, 196608)
    res["cpu_baseline"] = {
        "value": rate, "unit": "tokens/s", "cores": threads, "kind": "oracle",
        "sample": "%d random query rows of %d (both branches + gate), %.1f s, extrapolated to "
                  "whole tokens" % (rows, c.B * c.Hq * c.n, dt)}
    return res


if __name__ == "__main__":
    main()
