#!/usr/bin/env python
"""Benchmark of the Winograd convolution hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg3|cfg4|cfg2] [--points nova|half|std] [--workspace-mb M]

One "step" is one nova_conv2d_fwd call (input transform, transformed-domain
product, output transform) over one synthetic batch of the workload, with the
filter already transformed (as at inference time; that kernel is timed
separately and reported as filter_transform_ms).  Prints ONE JSON line.
With N > 1 (launched under torch.distributed.run) every rank runs its own batch
(weak scaling, no data-path collective); the time is the max over ranks.
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

METRIC = "fp16 Winograd conv TFLOP/s (direct-equivalent)"
UNIT = "TFLOP/s"


def read_peaks():
    """Measured peaks written by the driver, else the documented fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "tflops_burst": float(d["bf16_tflops"]),
                "tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.samples, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for s in self.samples:
            parts = [p.strip() for p in s.split(",")]
            if len(parts) < 6:
                continue
            try:
                mhz.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for nme, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(mhz)}


def workload(name):
    from synth import CONFIGS
    return CONFIGS[name]


FILTER_R = 3          # filter size of the run (--filter): 3, or 5 for the 5 x 5 extension


def flops(c):
    n = c.m + FILTER_R - 1
    th, tw = -(-c.H // c.m), -(-c.W // c.m)
    P = c.N * th * tw
    direct = 2.0 * c.N * c.H * c.W * c.K * c.C * FILTER_R * FILTER_R
    actual = 2.0 * n * n * c.K * c.C * P
    min_bytes = 2.0 * c.N * c.H * c.W * (c.C + c.K) + 2.0 * n * n * c.K * c.C
    return direct, actual, min_bytes, P


def _host_threads():
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1]))
    except Exception:
        return int(os.cpu_count() or 1)


def _oracle_sample(c, budget_s):
    """Inputs for a bounded sample: as many images of the batch as fit `budget_s` seconds."""
    from oracle import conv
    from synth import make_conv_inputs
    x, g = make_conv_inputs(1, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, c.seed, r=FILTER_R)
    conv.direct_conv_fp64(x, g)                      # page in BLAS
    t0 = time.perf_counter()
    conv.direct_conv_fp64(x, g)
    t1 = time.perf_counter() - t0
    n_img = int(max(1, min(c.N, budget_s / max(t1, 1e-4))))
    x, g = make_conv_inputs(n_img, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, c.seed, r=FILTER_R)
    return x, g, n_img


def time_oracle(c, budget_s=20.0):
    """The oracle's fp64 direct convolution (as it stands) on a bounded sample of the batch."""
    from oracle import conv
    x, g, n_img = _oracle_sample(c, budget_s / 3.0)
    best = float("inf")
    for _ in range(3):
        t0 = time.perf_counter()
        conv.direct_conv_fp64(x, g)
        best = min(best, time.perf_counter() - t0)
    fl = 2.0 * n_img * c.H * c.W * c.K * c.C * FILTER_R * FILTER_R
    return {"value": fl / best / 1e12, "unit": UNIT, "cores": _host_threads(), "kind": "oracle",
            "sample": "oracle.conv.direct_conv_fp64 (fp64, numpy) on %d of %d images of %s, best of 3"
                      % (n_img, c.N, c.name)}


def accuracy_report(c, nv, torch, n_img=2):
    """rel-L2 against the oracle's fp64 direct convolution, per point set of the workload, on the
    first n_img images (images are independent): the GPU path, and the oracle's rounding
    emulation of the same pipeline beside it.  Untimed."""
    import numpy as np
    from oracle import conv
    from synth import make_conv_inputs, point_set
    x, g = make_conv_inputs(n_img, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, c.seed, r=FILTER_R)
    y1 = conv.direct_conv_fp64(x, g)
    xd, gd = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
    from synth import pow2_range_scales
    rep = {}
    for kind in c.point_kinds:
        pts = point_set(kind, c.m + FILTER_R - 3)
        # each set as constructed, and with power-of-two row scales that normalise the range of
        # U and V (diagonal rescaling D_A D_G D_B = I; conditioning unchanged)
        for label, scaled in ((kind, False), (kind + "+pow2_rows", True)):
            sc = (None, None)
            if scaled:
                _, G, BT = nv.Plan(c.m, pts, nv.FP16_F32ACC, r=FILTER_R).matrices()
                sc = pow2_range_scales(G, BT)
            plan = nv.Plan(c.m, pts, nv.FP16_F32ACC, r=FILTER_R, scale_G=sc[0], scale_B=sc[1])
            y = plan.conv2d(xd, plan.filter_transform(gd))
            torch.cuda.synchronize()
            yh = y.cpu().numpy().astype(np.float32)
            e_gpu = conv.rel_l2(yh, y1)
            e_emu = conv.rel_l2(conv.winograd_conv_emulated(x, g, c.m, pts, "fp16", scales=sc), y1)
            kap, nrm = plan.kappa_matrices()
            rep[label] = {"kappa2_V": plan.kappa(), "kappa2_A_G_B": list(kap), "norm_product": nrm[0] * nrm[1] * nrm[2],
                          "rel_l2_gpu": e_gpu if np.isfinite(e_gpu) else None,
                          "rel_l2_emulation": e_emu if np.isfinite(e_emu) else None,
                          "nonfinite_outputs": int((~np.isfinite(yh)).sum())}
    return {"sample": "first %d images of %s" % (n_img, c.name), "points": rep}


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on the same workload and metric.
    Each step is one direct convolution of a bounded sample of the batch."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import conv
    c = workload(args.workload)
    x, g, n_img = _oracle_sample(c, min(6.0, 120.0 / (args.steps + args.warmup)))
    fl = 2.0 * n_img * c.H * c.W * c.K * c.C * FILTER_R * FILTER_R
    for _ in range(args.warmup):
        conv.direct_conv_fp64(x, g)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        conv.direct_conv_fp64(x, g)
    sec = (time.perf_counter() - t0) / args.steps
    val = fl / sec / 1e12
    sample = "oracle.conv.direct_conv_fp64 (fp64, numpy) on %d of %d images of %s per step" % (n_img, c.N, c.name)
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "%s: F(%dx%d,3x3), N=%d C=%d K=%d H=W=%d; %s"
                               % (c.name, c.m, c.m, c.N, c.C, c.K, c.H, sample)},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": _host_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def alu_ceiling(c, P, clocks):
    """Third ceiling beside tensor flops and HBM bytes: the fp32 arithmetic of the output transform,
    the one transform of the half pipeline that runs on the CUDA cores (the input transform is a
    tensor-core contraction).  Counted as executed for a point set symmetric about 0 - the +-pairs
    share their even / odd sums and the rows of 0 and infinity are copies - in fp32 lane-operations
    (an FMA, an add or a multiply on one value), against 128 lanes per SM per clock at the SM clock
    sampled during the run (the maximum clock if none was sampled)."""
    m, n = c.m, c.m + FILTER_R - 1
    q = (n - 2) // 2                                   # +-pairs
    row = 2 * q + m * q + 2                            # A^T applied to one row of M: sums/differences, m outputs, 2 copies added
    col = q * m * (2 + m) + 2 * m                      # per pair and column: sum, difference, m multiply-adds; rows 0 and infinity
    ops = n * row + col
    dense = m * n * n + m * m * n
    mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
    lanes = 148 * 128
    total = float(ops) * P * c.K
    return {"alu_us": total / (lanes * mhz * 1e6) * 1e6, "lane_ops_per_tile_filter": ops, "dense_lane_ops_per_tile_filter": dense,
            "sm_mhz": mhz, "kernel": "output transform (fp32, CUDA cores)"}


def run_fabric(args):
    """SM <-> L2 / HBM rates by access kind: a buffer that stays in L2 (48 MiB) and one that does
    not (1 GiB), all SMs and a quarter of them (per-SM against chip-wide limits)."""
    import torch
    import paper_2512_18453_b200 as nv
    from synth import point_set
    torch.cuda.set_device(0)
    plan = nv.Plan(2, point_set("std", 2))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    kinds = {0: "ld.global.v4", 1: "st.global.v4", 2: "half the warps load, half store", 3: "bulk copy global->shared",
             4: "bulk copy global->shared + st.global.v4", 5: "bulk copy shared->global",
             6: "bulk copy global->shared + shared->global"}
    rows = []
    for mib in (48, 1024):
        n = mib << 20
        src = torch.ones(n, dtype=torch.uint8, device="cuda")
        dst = torch.empty(n, dtype=torch.uint8, device="cuda")
        iters = 20 if mib == 48 else 2
        for ctas in (sms, sms // 4):
            for kind, label in kinds.items():
                for depth in ((4, 12) if kind in (3, 4, 6) else (1,)):
                    ms = plan.probe_fabric(kind, src, dst, iters=iters, ctas=ctas, depth=depth)
                    moved = n * iters * (2 if kind in (4, 6) else 1)
                    rows.append({"buffer_mib": mib, "ctas": ctas, "kind": label, "depth": depth if kind in (3, 4, 6) else None,
                                 "ms": ms, "tb_per_s": moved / (ms * 1e-3) / 1e12,
                                 "bytes_per_clk_per_sm_at_1965mhz": moved / (ms * 1e-3) / ctas / 1.965e9})
        del src, dst
    assert plan.device_status() == 0
    print(json.dumps({"fabric": rows}))


def run_wait_profile(args):
    """Where the warps of the transformed-domain product kernel spend their time: 20 calls of the
    workload with the wait-profiling variant of that kernel, the counters of the last one printed
    as shares of each warp role's total.  A measurement aid; its step time is not a bench value."""
    import torch
    import paper_2512_18453_b200 as nv
    from synth import point_set, make_conv_inputs
    torch.cuda.set_device(0)
    c = workload(args.workload)
    plan = nv.Plan(c.m, point_set(args.points, c.m), nv.FP16_F32ACC)
    x_np, g_np = make_conv_inputs(c.N, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, c.seed)
    x, g = torch.from_numpy(x_np).cuda(), torch.from_numpy(g_np).cuda()
    U = plan.filter_transform(g)
    y = torch.empty(c.N, c.H, c.W, c.K, dtype=torch.float16, device="cuda")
    ws = torch.empty(plan.workspace_bytes(c.N, c.H, c.W, c.C, c.K), dtype=torch.uint8, device="cuda")
    out = {}
    for name, flags in (("plain", 0), ("profiled", nv.PROFILE_WAITS)):
        for _ in range(5):
            plan.conv2d(x, U, y=y, workspace=ws, flags=flags)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(20):
            plan.conv2d(x, U, y=y, workspace=ws, flags=flags)
        e1.record()
        torch.cuda.synchronize()
        out["us_per_step_" + name] = e0.elapsed_time(e1) / 20 * 1e3
    w = plan.wait_profile()
    assert plan.device_status() == 0
    out["workload"] = c.name
    out["cycles_per_cta"] = w
    out["shares"] = {
        "producer_waiting_for_a_free_stage": w["producer_wait_stage"] / max(w["producer_total"], 1.0),
        "mma_waiting_for_operands": w["mma_wait_operands"] / max(w["mma_total"], 1.0),
        "mma_waiting_for_a_free_accumulator": w["mma_wait_accumulator"] / max(w["mma_total"], 1.0),
        "epilogue_waiting_for_an_accumulator": w["epilogue_wait_accumulator"] / max(w["epilogue_total"], 1.0),
        "epilogue_storing": 1.0 - w["epilogue_wait_accumulator"] / max(w["epilogue_total"], 1.0),
    }
    print(json.dumps({"wait_profile": out}))


def rank_seed(base_seed, rank):
    """Each rank draws its own batch (weak scaling): the seed is offset by the rank."""
    return base_seed + 100 * rank


def max_over_ranks(ms, dist, device):
    """The slowest rank's time; `dist` is torch.distributed or None for one process."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, direct_flops_per_rank, ms_per_step):
    """Aggregate direct-equivalent TFLOP/s of all ranks (each processed its own batch)."""
    return world * direct_flops_per_rank / (ms_per_step * 1e-3) / 1e12


def run_ours(args):
    import numpy as np
    import torch
    import paper_2512_18453_b200 as nv
    from synth import point_set, make_conv_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    c = workload(args.workload)
    if args.images:                                  # profiling aid: a smaller batch of the same layer
        import dataclasses
        c = dataclasses.replace(c, N=args.images, name="%s[N=%d]" % (c.name, args.images))
    n_points = c.m + 2
    if FILTER_R == 5:                                # same number of points, tile smaller by two
        import dataclasses
        c = dataclasses.replace(c, m=c.m - 2, name="%s[5x5,F(%d,5)]" % (c.name, c.m - 2))
    direct, actual, min_bytes, P = flops(c)
    pts = point_set(args.points, n_points - 2)
    plan = nv.Plan(c.m, pts, nv.FP16_F32ACC, r=FILTER_R)
    # each rank gets its own batch (weak scaling): seed offset by rank
    x_np, g_np = make_conv_inputs(c.N, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, rank_seed(c.seed, rank),
                                  r=FILTER_R)
    g = torch.from_numpy(g_np).cuda()
    n_sets = 3
    xs = [torch.from_numpy(x_np).cuda() if i == 0 else torch.from_numpy(np.roll(x_np, i, axis=0)).cuda()
          for i in range(n_sets)]
    ys = [torch.empty(c.N, c.H, c.W, c.K, dtype=torch.float16, device="cuda") for _ in range(n_sets)]
    ws_bytes = plan.workspace_bytes(c.N, c.H, c.W, c.C, c.K) if args.workspace_mb is None \
        else int(args.workspace_mb * (1 << 20))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    flags = {"auto": 0, "tcgen05": nv.GEMM_TCGEN05, "simt": nv.GEMM_SIMT}[args.gemm]
    launches = plan.launch_count(c.N, c.H, c.W, c.C, c.K, ws_bytes, flags)

    # S1, once per layer: timed on its own
    U = plan.filter_transform(g)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        U = plan.filter_transform(g)
    e1.record()
    torch.cuda.synchronize()
    filter_ms = e0.elapsed_time(e1) / 5

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing.  One step = one nova_conv2d_fwd call; with --launch graph
    # (default) each buffer set's call is captured once into a CUDA graph and the timed loop
    # replays the graphs, so that the host's per-launch work does not pace the device.
    def step_direct(i):
        plan.conv2d(xs[i % n_sets], U, y=ys[i % n_sets], workspace=ws, flags=flags)

    step = step_direct
    step_direct(0)
    torch.cuda.synchronize()
    if args.launch == "graph":
        graphs = []
        side = torch.cuda.Stream()
        for i in range(n_sets):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(gr, stream=side):
                    step_direct(i)
            graphs.append(gr)
        torch.cuda.synchronize()

        def step(i):
            graphs[i % n_sets].replay()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    total_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
    ms_per_step = total_ms / args.steps
    status = plan.device_status()

    # ---- spread of single steps: 100 steps timed one by one (an event pair each), median and minimum
    n_single = min(100, args.steps)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_single)]
    for i, (a0, a1) in enumerate(evs):
        a0.record()
        step(i)
        a1.record()
    torch.cuda.synchronize()
    singles = sorted(a0.elapsed_time(a1) for a0, a1 in evs)
    step_stats = {"n": n_single, "median_us": 1e3 * singles[len(singles) // 2], "min_us": 1e3 * singles[0],
                  "note": "single steps between their own event pairs; the headline ms_per_step is the mean of the back-to-back run"}

    # ---- per-kernel durations (events around each kernel, same steps, separate pass)
    kms = [0.0, 0.0, 0.0]
    prof_steps = min(args.steps, 20)
    for i in range(prof_steps):
        t = plan.conv2d_timed(xs[i % n_sets], U, ys[i % n_sets], ws, flags=flags)
        kms = [a + b for a, b in zip(kms, t)]
    kms = [v / prof_steps for v in kms]
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: host buffers in and out through the C ABI
    xh = torch.from_numpy(x_np).pin_memory()
    yh = torch.empty(c.N, c.H, c.W, c.K, dtype=torch.float16).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        plan.conv2d_host(xh, U, yh, xs[0], ys[0], ws, flags=flags)
    barrier()
    e0.record()
    for i in range(e2e_steps):
        plan.conv2d_host(xh, U, yh, xs[i % n_sets], ys[i % n_sets], ws, flags=flags)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / e2e_steps

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = read_peaks()
    chunks = launches // 3
    names = ["input_transform", "product_tcgen05" if flags != nv.GEMM_SIMT else "product_simt", "output_transform"]
    n2 = (c.m + FILTER_R - 1) ** 2
    elt = 2
    # algorithmic bytes / flops per step of each kernel class
    alg = [
        ("hbm", 2.0 * c.N * c.H * c.W * c.C + elt * n2 * P * c.C),        # read x, write V
        ("tensor", actual),                                                # 2 n^2 K C P flop
        ("hbm", 4.0 * n2 * P * c.K + 2.0 * c.N * c.H * c.W * c.K),         # read M, write y
    ]
    dom = max(range(3), key=lambda i: kms[i])
    bound, work = alg[dom]
    dur_launch = kms[dom] * 1e-3 / chunks
    if bound == "tensor":
        achieved, peak, runit = work / chunks / dur_launch / 1e12, peaks["tflops_burst"], "TFLOP/s"
    else:
        achieved, peak, runit = work / chunks / dur_launch / 1e9, peaks["hbm_gbs"], "GB/s"
    # DRAM bytes per launch come from an ncu capture, which this run is not: null here
    traffic = None
    alu = alu_ceiling(c, P, clocks)
    roof_s = max(actual / (peaks["tflops_burst"] * 1e12), min_bytes / (peaks["hbm_gbs"] * 1e9))
    value = whole_job_value(world, direct, ms_per_step)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 (f32 accumulate)", "data": "synthetic",
        "config": {
            "workload": "%s: F(%dx%d,%dx%d) %s points, N=%d C=%d K=%d H=W=%d per GPU, NHWC, ReLU'd N(0,1) x He-normal"
                        % (c.name, c.m, c.m, FILTER_R, FILTER_R, args.points, c.N, c.C, c.K, c.H),
            "step": "nova_conv2d_fwd (input transform, tcgen05 product, output transform); filter transform once per layer",
            "l2": "inputs/outputs rotate over %d buffer sets (%.0f MB > 126 MB L2)" % (n_sets, n_sets * (x_np.nbytes + ys[0].numel() * 2) / 1e6),
            "workspace_mb": ws_bytes / (1 << 20), "chunks": chunks, "gemm": args.gemm,
            "launch": "CUDA graph replay of the step's kernels" if args.launch == "graph" else "direct launches",
        },
        "tflops_actual": world * actual / (ms_per_step * 1e-3) / 1e12,
        "path_roofline": {"roofline_us": roof_s * 1e6, "achieved_us": ms_per_step * 1e3,
                          "frac": roof_s / (ms_per_step * 1e-3), "peaks": peaks["source"],
                          "tensor_us": actual / (peaks["tflops_burst"] * 1e12) * 1e6,
                          "hbm_us": min_bytes / (peaks["hbm_gbs"] * 1e9) * 1e6,
                          "alu_us": alu["alu_us"], "alu": alu},
        "kernels_ms_per_step": {n_: v for n_, v in zip(names, kms) if n_ != "-"},
        "single_step": step_stats,
        "filter_transform_ms": filter_ms,
        "roofline": {"kernel": names[dom], "bound": bound, "achieved": achieved, "peak": peak, "unit": runit,
                     "frac": achieved / peak, "traffic": traffic,
                     "traffic_note": "null: DRAM counters are taken under ncu, never in a timed run",
                     "peak_source": peaks["source"], "launch_us": dur_launch * 1e6},
        "e2e": {"value": world * direct / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(x_np.nbytes), "d2h_bytes_per_step": int(yh.numel() * 2)},
        "gpu_launches": launches * args.steps,
        "device_status": status,
        "kappa2_V": plan.kappa(),
        "clocks": clocks,
    }
    if world == 1 and (args.accuracy or not args.no_cpu_baseline):
        out["accuracy"] = accuracy_report(c, nv, torch)
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = time_oracle(c)
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def run_int8(args):
    """The INT8 Winograd-domain pipeline on the same workloads: one step = one
    nova_conv2d_fwd_int8 call (quantising input transform - two passes when the scale of V is
    derived from the data -, kind::i8 tensor-core product, dequantising output transform)."""
    import numpy as np
    import torch
    import paper_2512_18453_b200 as nv
    from synth import point_set, make_conv_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    c = workload(args.workload)
    if args.images:
        import dataclasses
        c = dataclasses.replace(c, N=args.images, name="%s[N=%d]" % (c.name, args.images))
    n_points = c.m + 2
    if FILTER_R == 5:                                # same number of points, tile smaller by two
        import dataclasses
        c = dataclasses.replace(c, m=c.m - 2, name="%s[5x5,F(%d,5)]" % (c.name, c.m - 2))
    direct, actual, _, P = flops(c)
    n2 = n_points ** 2
    min_bytes = 2.0 * c.N * c.H * c.W * (c.C + c.K) + 1.0 * n2 * c.K * c.C
    pts = point_set(args.points, n_points - 2)
    coef = nv.COEF_FP32 if args.int8_coef == "fp32" else nv.COEF_ROUND_TO_MODE
    plan = nv.Plan(c.m, pts, nv.FP16_F32ACC, coef, r=FILTER_R)
    quant = nv.QUANT_PER_CHANNEL if args.int8_quant == "per_channel" else nv.QUANT_PER_TENSOR
    x_np, g_np = make_conv_inputs(c.N, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, rank_seed(c.seed, rank),
                                  r=FILTER_R)
    g = torch.from_numpy(g_np).cuda()
    n_sets = 3
    xs = [torch.from_numpy(np.roll(x_np, i, axis=0)).cuda() for i in range(n_sets)]
    ys = [torch.empty(c.N, c.H, c.W, c.K, dtype=torch.float16, device="cuda") for _ in range(n_sets)]
    ws = torch.empty(plan.int8_workspace_bytes(c.N, c.H, c.W, c.C, c.K), dtype=torch.uint8, device="cuda")
    Uq, sU = plan.filter_transform_int8(g, quant)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        Uq, sU = plan.filter_transform_int8(g, quant)
    e1.record()
    torch.cuda.synchronize()
    filter_ms = e0.elapsed_time(e1) / 5
    scale_V = 0.0
    if args.int8_static_scale:                      # calibrate once on the first buffer set
        plan.conv2d_int8(xs[0], Uq, sU, 0.0, y=ys[0], workspace=ws)
        torch.cuda.synchronize()
        scale_V = float(ws[:4].view(torch.float32).item())

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def step_direct(i):
        plan.conv2d_int8(xs[i % n_sets], Uq, sU, scale_V, y=ys[i % n_sets], workspace=ws)

    step = step_direct
    step_direct(0)
    torch.cuda.synchronize()
    if args.launch == "graph":
        graphs = []
        side = torch.cuda.Stream()
        for i in range(n_sets):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(gr, stream=side):
                    step_direct(i)
            graphs.append(gr)
        torch.cuda.synchronize()

        def step(i):
            graphs[i % n_sets].replay()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    ms_per_step = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / args.steps
    status = plan.device_status()
    kms = [0.0] * 4
    prof_steps = min(args.steps, 20)
    for i in range(prof_steps):
        _, t = plan.conv2d_int8(xs[i % n_sets], Uq, sU, scale_V, y=ys[i % n_sets], workspace=ws, timed=True)
        kms = [a + b for a, b in zip(kms, t)]
    kms = [v / prof_steps for v in kms]
    clocks = sampler.stop() if rank == 0 else None

    # end to end: pinned host input in, host output back, around the C-ABI call
    xh = torch.from_numpy(x_np).pin_memory()
    yh = torch.empty(c.N, c.H, c.W, c.K, dtype=torch.float16).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step(i):
        xs[i % n_sets].copy_(xh, non_blocking=True)
        plan.conv2d_int8(xs[i % n_sets], Uq, sU, scale_V, y=ys[i % n_sets], workspace=ws)
        yh.copy_(ys[i % n_sets], non_blocking=True)
    for i in range(2):
        e2e_step(i)
    barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / e2e_steps
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = read_peaks()
    passes = 1 if scale_V > 0 else 2
    names = ["input_transform_int8 (%d pass%s)" % (passes, "" if passes == 1 else "es"), "product_tcgen05_i8",
             "output_transform_dequant"]
    # algorithmic work per step of each kernel class; the int8 tensor peak is twice the measured
    # bf16 one (nominal ratio of the dense peaks)
    alg = [("hbm", passes * 2.0 * c.N * c.H * c.W * c.C + 1.0 * n2 * P * c.C),
           ("tensor", actual),
           ("hbm", 4.0 * n2 * P * c.K + 2.0 * c.N * c.H * c.W * c.K)]
    dom = max(range(3), key=lambda i: kms[i])
    bound, work = alg[dom]
    dur = kms[dom] * 1e-3
    i8_peak = 2.0 * peaks["tflops_burst"]
    if bound == "tensor":
        achieved, peak, runit = work / dur / 1e12, i8_peak, "TOP/s"
    else:
        achieved, peak, runit = work / dur / 1e9, peaks["hbm_gbs"], "GB/s"
    roof_s = max(actual / (i8_peak * 1e12), min_bytes / (peaks["hbm_gbs"] * 1e9))
    out = {
        "metric": METRIC.replace("fp16", "int8"), "value": whole_job_value(world, direct, ms_per_step), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "s8 (s32 accumulate)",
        "data": "synthetic",
        "config": {
            "workload": "%s: F(%dx%d,%dx%d) %s points, N=%d C=%d K=%d H=W=%d per GPU, NHWC, ReLU'd N(0,1) x He-normal"
                        % (c.name, c.m, c.m, FILTER_R, FILTER_R, args.points, c.N, c.C, c.K, c.H),
            "step": "nova_conv2d_fwd_int8 (%s scale of U, %s scale of V, %s coefficient tables)"
                    % (args.int8_quant, "static" if scale_V > 0 else "data-derived", args.int8_coef),
            "l2": "inputs/outputs rotate over %d buffer sets (%.0f MB > 126 MB L2)"
                  % (n_sets, n_sets * (x_np.nbytes + ys[0].numel() * 2) / 1e6),
            "launch": "CUDA graph replay of the step's kernels" if args.launch == "graph" else "direct launches",
        },
        "tops_actual": world * actual / (ms_per_step * 1e-3) / 1e12,
        "path_roofline": {"roofline_us": roof_s * 1e6, "achieved_us": ms_per_step * 1e3,
                          "frac": roof_s / (ms_per_step * 1e-3), "peaks": peaks["source"] + "; int8 tensor peak = 2 x bf16"},
        "kernels_ms_per_step": dict(zip(names, kms[:3])),
        "filter_transform_ms": filter_ms,
        "roofline": {"kernel": names[dom], "bound": bound, "achieved": achieved, "peak": peak, "unit": runit,
                     "frac": achieved / peak, "traffic": None, "peak_source": peaks["source"], "launch_us": dur * 1e6},
        "e2e": {"value": world * direct / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(x_np.nbytes), "d2h_bytes_per_step": int(yh.numel() * 2)},
        "gpu_launches": (3 + 2 * passes) * args.steps if scale_V == 0 else 4 * args.steps,
        "device_status": status, "kappa2_V": plan.kappa(), "clocks": clocks,
    }
    if world == 1 and (args.accuracy or not args.no_cpu_baseline):
        out["accuracy"] = accuracy_report_int8(c, nv, torch, coef, args.int8_coef)
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = time_oracle(c)
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def accuracy_report_int8(c, nv, torch, coef, coef_name, n_img=2):
    """rel-L2 of the INT8 pipeline against the fp64 direct convolution per point set, per-tensor and
    per-channel, with and without power-of-two range scaling; the oracle's emulation beside it."""
    import numpy as np
    from oracle import conv
    from synth import make_conv_inputs, point_set, pow2_range_scales
    x, g = make_conv_inputs(n_img, c.H, c.W, c.C, c.K, c.dtype, c.relu_inputs, c.he_weights, c.seed, r=FILTER_R)
    y1 = conv.direct_conv_fp64(x, g)
    xd, gd = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
    rep = {}
    for kind in c.point_kinds:
        pts = point_set(kind, c.m + FILTER_R - 3)
        _, G, BT = nv.Plan(c.m, pts, nv.FP16_F32ACC, r=FILTER_R).matrices()
        for label, sc in ((kind, (None, None)), (kind + "+pow2_rows", pow2_range_scales(G, BT))):
            plan = nv.Plan(c.m, pts, nv.FP16_F32ACC, coef, r=FILTER_R, scale_G=sc[0], scale_B=sc[1])
            for qname, quant in (("per_tensor", nv.QUANT_PER_TENSOR), ("per_channel", nv.QUANT_PER_CHANNEL)):
                Uq, sU = plan.filter_transform_int8(gd, quant)
                y = plan.conv2d_int8(xd, Uq, sU, 0.0)
                torch.cuda.synchronize()
                yh = y.cpu().numpy().astype(np.float32)
                e_gpu = conv.rel_l2(yh, y1)
                e_emu = conv.rel_l2(conv.winograd_conv_int8_emulated(
                    x, g, c.m, pts, per_channel=(qname == "per_channel"),
                    coef="fp32" if coef_name == "fp32" else "mode", scales=sc), y1)
                rep["%s/%s" % (label, qname)] = {
                    "kappa2_V": plan.kappa(), "rel_l2_gpu": e_gpu if np.isfinite(e_gpu) else None,
                    "rel_l2_emulation": e_emu if np.isfinite(e_emu) else None,
                    "nonfinite_outputs": int((~np.isfinite(yh)).sum())}
    return {"sample": "first %d images of %s" % (n_img, c.name), "points": rep}


def run_vgg(args):
    """cfg5: the 13 convolution layers of VGG-16 (ReLU in the epilogue, 2x2 max-pool between the
    blocks) on a synthetic 224x224 batch, F(8,3) NOVA points unless --points says otherwise.
    A step = the whole stack; reports images/s beside the direct-equivalent TFLOP/s."""
    import numpy as np
    import torch
    import paper_2512_18453_b200 as nv
    from synth import point_set, make_vgg_inputs, VGG16_LAYERS
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("--workload cfg5 is a single-GPU report")
    torch.cuda.set_device(0)
    N = args.images or 32
    m = args.tile
    pts = point_set(args.points, m)
    plan = nv.Plan(m, pts, nv.FP16_F32ACC)
    x_np, weights = make_vgg_inputs(N)
    x = torch.from_numpy(x_np).cuda()
    Us = [plan.filter_transform(torch.from_numpy(w).cuda()) for w in weights]
    flags = nv.RELU
    # buffers: activations of every layer, one scratch sized for the largest layer
    shapes, hw, c_in = [], 224, 8
    for (ci, co, pool) in VGG16_LAYERS:
        shapes.append((hw, max(ci, 8), co, pool))
        hw = hw // 2 if pool else hw
    ws_bytes = max(plan.workspace_bytes(N, h, h, ci, co) for (h, ci, co, _) in shapes) if args.workspace_mb is None \
        else int(args.workspace_mb * (1 << 20))
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    ys = [None if pool else torch.empty(N, h, h, co, dtype=torch.float16, device="cuda") for (h, ci, co, pool) in shapes]
    ps = [torch.empty(N, h // 2, h // 2, co, dtype=torch.float16, device="cuda") if pool else None
          for (h, ci, co, pool) in shapes]
    L = nv.lib()

    def step():
        # the 2 x 2 max-pool after a block's last convolution is fused into that layer's output
        # transform (NOVA_POOL2X2): the unpooled activations are never written
        a = x
        for i, (h, ci, co, pool) in enumerate(shapes):
            if pool:
                plan.conv2d(a, Us[i], y=ps[i], workspace=ws, flags=flags | nv.POOL2X2)
                a = ps[i]
            else:
                plan.conv2d(a, Us[i], y=ys[i], workspace=ws, flags=flags)
                a = ys[i]
        return a

    out_t = step()
    torch.cuda.synchronize()
    gr = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(gr, stream=side):
            step()
    torch.cuda.synchronize()
    for _ in range(args.warmup):
        gr.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.1)
    steps = min(args.steps, 200)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        gr.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    clocks = sampler.stop()
    status = plan.device_status()
    # per-layer durations: the layer's call five times back to back between two events (direct launches;
    # the activations of the last step are still in the buffers, so every layer sees its real input)
    reps = 5
    layers_ms = []
    a = x
    for i, (h, ci, co, pool) in enumerate(shapes):
        e0l, e1l = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fl, out_i = (flags | nv.POOL2X2, ps[i]) if pool else (flags, ys[i])
        plan.conv2d(a, Us[i], y=out_i, workspace=ws, flags=fl)
        e0l.record()
        for _ in range(reps):
            plan.conv2d(a, Us[i], y=out_i, workspace=ws, flags=fl)
        e1l.record()
        torch.cuda.synchronize()
        layers_ms.append("%dx%d C%d K%d: %.3f" % (h, h, ci, co, e0l.elapsed_time(e1l) / reps))
        a = ps[i] if pool else ys[i]
    direct = sum(2.0 * N * h * h * co * ci_true * 9 for (h, _, co, _), (ci_true, _, _) in zip(shapes, VGG16_LAYERS))
    launches = sum(plan.launch_count(N, h, h, ci, co, ws_bytes, flags) for (h, ci, co, _) in shapes)
    # accuracy on the first two images (images are independent), untimed
    acc = None
    if not args.no_cpu_baseline:
        from oracle import conv
        x2, _ = x_np[:2], None
        ref = conv.vgg_stack_fp64(x2, weights, VGG16_LAYERS)
        emu = conv.vgg_stack_emulated(x2, weights, VGG16_LAYERS, m, pts)
        got = out_t[:2].cpu().numpy()
        acc = {"sample": "first 2 images", "rel_l2_gpu": conv.rel_l2(got, ref), "rel_l2_emulation": conv.rel_l2(emu, ref)}
    out = {
        "metric": METRIC, "value": direct / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 (f32 accumulate)", "data": "synthetic",
        "config": {"workload": "cfg5: VGG-16 conv stack, 13 layers, N=%d, 224x224x3 (padded to 8 channels), F(%dx%d,3x3) %s points"
                               % (N, m, m, args.points),
                   "step": "13 x nova_conv2d_fwd (ReLU fused; the 5 max-pools fused into the output transforms), CUDA graph replay",
                   "workspace_mb": ws_bytes / (1 << 20)},
        "images_per_s": N / (ms * 1e-3), "layers_ms": layers_ms, "gpu_launches": launches * steps, "device_status": status,
        "accuracy": acc, "clocks": clocks,
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--tile", type=int, default=8, help="tile size m of the cfg5 stack")
    ap.add_argument("--points", default="nova")
    ap.add_argument("--gemm", default="auto", choices=["auto", "tcgen05", "simt"])
    ap.add_argument("--workspace-mb", type=float, default=None)
    ap.add_argument("--launch", default="graph", choices=["graph", "direct"])
    ap.add_argument("--fabric", action="store_true",
                    help="measure the SM <-> L2 / HBM rates by access kind (nova_probe_fabric) and print them")
    ap.add_argument("--wait-profile", action="store_true",
                    help="print where the product kernel's warps wait (NOVA_PROFILE_WAITS; not a bench value)")
    ap.add_argument("--images", type=int, default=0, help="override the batch size (profiling aid)")
    ap.add_argument("--accuracy", action="store_true",
                    help="report rel-L2 per point set (and per rescaled variant) even with --no-cpu-baseline")
    ap.add_argument("--filter", type=int, default=3, choices=[3, 5],
                    help="filter size: 5 runs the 5 x 5 extension on the same layer with the tile two smaller (same points)")
    ap.add_argument("--int8", action="store_true", help="time the INT8 Winograd-domain pipeline instead")
    ap.add_argument("--int8-quant", default="per_tensor", choices=["per_tensor", "per_channel"])
    ap.add_argument("--int8-coef", default="half", choices=["half", "fp32"],
                    help="coefficient tables: half-rounded (tensor-core input transform) or float32 (CUDA cores)")
    ap.add_argument("--int8-static-scale", action="store_true",
                    help="calibrate the scale of V once instead of deriving it from every batch")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    global FILTER_R
    FILTER_R = args.filter
    if args.impl == "reference":
        run_reference(args)
    elif args.fabric:
        run_fabric(args)
    elif args.wait_profile:
        run_wait_profile(args)
    elif args.workload == "cfg5":
        run_vgg(args)
    elif args.int8:
        run_int8(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
