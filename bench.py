#!/usr/bin/env python
"""Benchmark of the packed low-bit convolution path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra]
                    [--workload c2|c3|c4|c5] [--algo packed|unpacked|dp4a|emu64]

A "step" is one pass of the whole hot path over the 1-D bitwidth sweep: 48 full convolutions of a
2^24-element signal (p = q = 1..8, K in {3,5,7}, unsigned and signed), each launch reading its own
16 MiB input and writing its own 64 MiB int32 output, so a step streams about 3.9 GB and nothing
is served from L2.  The metric is effective multiply-accumulates of the plain definition per
second.  The line also carries the roofline of the dominant kernel, the same path timed end to
end from pinned host buffers, the oracle timed on the host cores, and (unless --no-extra) the
2-D layer and full-network workloads with the one-product-per-multiply comparator beside them.
"""
from __future__ import annotations

import argparse
import hashlib
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

METRIC = "effective low-bit conv MAC/s"
UNIT = "MAC/s"
HBM_FALLBACK_GBS = 6650.0            # earlier pool measurement, used only when MEASURED_PEAKS.json is absent
# Integer multiply-add lanes per SM per clock, measured with shared-memory-fed operands: the 32-bit
# multiply-add of the comparator issues on 64 lanes, the 32x32->64 multiply with 64-bit accumulate of
# the packed kernels on 32.
IMAD32_PER_CLK_PER_SM = 64
IMAD_WIDE_PER_CLK_PER_SM = 32
TABLE_REPEATS = 7                    # timed repeats per cell of the per-case table (median and max - min are reported)

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the last ncu capture of the kernel: six
# consecutive launches of the p=q=4, K=3 signed case at 2^24 rotating over three input and three output
# buffers, caches not flushed between launches (steady state): 12.5-13.4 MB read, 62.9-66.1 MB written
# (the 8-bit K=7 case: 79.9 MB in all).  (With the caches flushed before each launch the same kernel shows
# 16.8 MB read and 8-9 MB written: most of a launch's output is then still in the 126 MB L2 when its
# counters stop.)  The SHA-256 values are those of the kernel sources at capture time; a changed source voids
# the figure.
NCU_TRAFFIC = {
    "conv1d_bs": {"sha256": "36e8f9ed30e2667834955a0cfb06cb0462a71beae17cbcfc024e007a0ee74fd9",
                  "sha256_run": "322f9167bd95031f2841bdd2e540d4bd24431054ad2d45e0ce1474457f5564c2",
                  "bytes_per_output": (13.08e6 + 65.07e6) / 16777218.0},
}


# Warp instructions one launch of the packed layer kernel executes (smsp__inst_executed.sum of the captures behind
# profiles/conv2d_kernel_c3.txt and _c4.txt), for the issue model of the 2-D rooflines; void when the source changes.
NCU_INSTRUCTIONS = {
    "c3": {"sha256": "dd5f48402620b0de3ccab755f40e1210a87800596c3d25131297b506941b6beb", "warp_instructions": 41575448.0},
    "c4": {"sha256": "dd5f48402620b0de3ccab755f40e1210a87800596c3d25131297b506941b6beb", "warp_instructions": 87595968.0},
}


def _source_hash(name: str) -> str:
    with open(os.path.join(ROOT, "paper_2208_00763_b200", "csrc", name), "rb") as fh:
        return hashlib.sha256(fh.read()).hexdigest()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), float(d.get("sm_max_mhz", 1965.0)), "measured"
    return HBM_FALLBACK_GBS, 1965.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def keep_busy_until_sampled(self, run_step, synchronize, min_samples: int = 2, timeout_s: float = 3.0):
        """The timed region can be shorter than nvidia-smi's first sampling period: keep the same steps running,
        untimed, until the sampler has seen the GPU under this load."""
        if self.proc is None:
            return
        t0 = time.time()
        while len(self.lines) < min_samples and time.time() - t0 < timeout_s:
            run_step()
            synchronize()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [t.strip() for t in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
# reference arm and CPU baseline: the oracle as it stands, on the host cores
# ----------------------------------------------------------------------------------------------

def oracle_inputs(sample_len: int, seed_offset: int = 0, compact: bool = False):
    """The 48 sweep cases as code values; `compact` keeps them as int16 (the oracle widens them itself), so that the
    full-length sweep fits in 1.6 GB of host memory."""
    import numpy as np
    from paper_2208_00763_b200 import inputs
    data = []
    for case in inputs.c2_cases(sample_len):
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"],
                                  case["seed"] + seed_offset)
        data.append((f.astype(np.int16) if compact else f, g))
    return data


def oracle_sweep(data):
    """One pass of the sweep through the oracle (int64 direct convolution).  Returns (MACs, seconds)."""
    from oracle import direct
    macs = 0.0
    t0 = time.perf_counter()
    for f, g in data:
        direct.conv1d_full(f, g)
        macs += float(f.size + g.size - 1) * g.size
    return macs, time.perf_counter() - t0


def inputs_mod():
    from paper_2208_00763_b200 import inputs
    return inputs


def cpu_baseline(sample_len: int):
    """The oracle as it stands on the host cores: the 48 sweep cases at `sample_len`, repeated for about 10 s."""
    from oracle import direct
    data = oracle_inputs(sample_len)
    oracle_sweep(data[:2])
    macs, secs, passes = 0.0, 0.0, 0
    while secs < 10.0 and passes < 400:
        m, s = oracle_sweep(data)
        macs += m
        secs += s
        passes += 1
    # the definition on one thread: one pass over the same sample
    threads_all = direct.num_threads()
    direct.set_num_threads(1)
    m1, s1 = oracle_sweep(data)
    direct.set_num_threads(threads_all)
    layers = {}
    for name, shape, batch in (("c3", inputs_mod().C3_SHAPE, 2), ("c4", inputs_mod().C4_SHAPE, 2)):
        x, w = inputs_mod().layer_case(shape, batch=batch)
        t0 = time.perf_counter()
        direct.conv2d_nchw(x, w, shape["pad"])
        dt = time.perf_counter() - t0
        Ho = shape["H"] + 2 * shape["pad"] - shape["K"] + 1
        lm = float(batch) * shape["Co"] * Ho * Ho * shape["Ci"] * shape["K"] ** 2
        layers[name] = {"value": lm / dt, "unit": UNIT, "sample": "%d of %d images, %.2f s" % (batch, shape["B"], dt)}
    # the paper's own CPU experiment on this host: its packed loop (Algorithm 2) beside the plain loops,
    # one thread, K = 3, where the kernel fits one 32-bit word
    from oracle import algorithm2
    alg2 = {}
    rng_len = 1 << 22
    threads_before = direct.num_threads()
    direct.set_num_threads(1)
    for bits in (1, 2, 4):
        for signed in (False, True):
            if algorithm2.layout(bits, bits, 3, signed) is None:
                continue
            f, g = inputs_mod().conv1d_case(rng_len, 3, bits, bits, signed, signed, 7000 + 10 * bits + int(signed))
            t0 = time.perf_counter()
            direct.conv1d_full(f, g)
            t1 = time.perf_counter()
            algorithm2.conv1d_full(f, g, bits, bits, signed, 1)
            t2 = time.perf_counter()
            alg2["p%d_%s" % (bits, "s" if signed else "u")] = {"plain_ms": 1e3 * (t1 - t0), "packed_ms": 1e3 * (t2 - t1),
                                                             "speedup": (t1 - t0) / (t2 - t1)}
    direct.set_num_threads(threads_before)
    return {"value": macs / secs, "unit": UNIT, "cores": direct.num_threads(), "kind": "oracle", "layers": layers,
            "one_thread": {"value": m1 / s1, "unit": UNIT, "sample": "one pass over the same 48 cases, %.1f s" % s1},
            "algorithm2_one_thread": alg2,
            "sample": "%d pass(es) over the 48 sweep cases at signal length %d (benchmark length 2^24), int64 direct "
                      "convolution, OpenMP over outputs, %.1f s of CPU time" % (passes, sample_len, secs)}


def run_reference(args):
    from paper_2208_00763_b200 import ranks
    if ranks.rank_info()[1] != 0:
        return 0                      # the oracle runs once, on rank 0's host cores
    from oracle import direct
    sample_len = args.length                      # the benchmark's own signal length (2^24 unless --length says otherwise)
    data = oracle_inputs(sample_len, compact=True)
    for _ in range(args.warmup):
        oracle_sweep(data[:4])
    total_macs, total_secs = 0.0, 0.0
    for _ in range(args.steps):
        m, s = oracle_sweep(data)
        total_macs += m
        total_secs += s
    value = total_macs / total_secs
    sample = "each step: the 48 sweep cases at signal length %d (the benchmark's configuration), one case after the other" % sample_len
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_secs / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int64", "data": "synthetic",
        "config": {"workload": "c2: 1-D bitwidth sweep, %d full convolutions of length 2^%d (p=q=1..8, K=3/5/7, unsigned+signed), "
                               "int8-stored codes in, int32 out" % (len(data), sample_len.bit_length() - 1),
                   "oracle": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": direct.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------

def run_ours(args):
    import numpy as np
    import torch

    from paper_2208_00763_b200 import binding as hk
    from paper_2208_00763_b200 import inputs, network, ranks

    world, rank, local_rank = ranks.rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ranks.init("nccl", dev)
    hk.lib()
    hbm_peak_gbs, sm_max_mhz, peak_kind = measured_peaks()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    # multiply-adds per second by kind of multiply
    imad_peak = {"packed": sms * IMAD_WIDE_PER_CLK_PER_SM * sm_max_mhz * 1e6,
                 "unpacked": sms * IMAD32_PER_CLK_PER_SM * sm_max_mhz * 1e6}

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms: float) -> float:
        return ranks.max_over_ranks(ms, dev)

    # measured integer-pipe rates (register-only kernels of the library), the denominators of the "alu" rooflines
    peaks = None
    if rank == 0:
        peaks = {}
        for kind in ("mad_wide_u32", "mad_wide_s32", "mad_lo_s32", "logic", "shift", "prmt", "mad_wide_with_logic"):
            r = hk.pipe_rate(kind, iters=2048, device=dev)
            peaks[kind] = {"T_per_s": r["ops_per_second"] / 1e12, "lanes_per_clk_per_sm_at_max_clock": r["lanes_per_clock_per_sm"]}
        peaks["derived"] = {"mad_wide_T_per_s": imad_peak["packed"] / 1e12, "mad_lo_T_per_s": imad_peak["unpacked"] / 1e12,
                            "how": "SMs x lanes/clk x max SM clock (%d SMs, %d / %d lanes, %.0f MHz)"
                                   % (sms, IMAD_WIDE_PER_CLK_PER_SM, IMAD32_PER_CLK_PER_SM, sm_max_mhz)}
        # scheduler cycles per warp-wide multiply-add = 128 / (lanes per clock and SM); the mixed kernel issues one logic
        # instruction per two multiply-adds, so twice the difference is what one such instruction costs the multiply stream
        pure, mixed = (peaks[k]["lanes_per_clk_per_sm_at_max_clock"] for k in ("mad_wide_u32", "mad_wide_with_logic"))
        peaks["issue_model"] = {"cycles_per_wide_multiply_add": 128.0 / pure,
                                "cycles_added_per_other_instruction": 2.0 * (128.0 / mixed - 128.0 / pure)}
        imad_peak["issue"] = dict(peaks["issue_model"], schedulers=4 * sms, clock_hz=sm_max_mhz * 1e6)
        imad_peak["packed_measured"] = max(peaks["mad_wide_u32"]["T_per_s"], peaks["mad_wide_s32"]["T_per_s"]) * 1e12
        imad_peak["unpacked_measured"] = peaks["mad_lo_s32"]["T_per_s"] * 1e12

    # ---- the sweep: every rank runs the whole sweep on its own data (weak scaling, no exchange)
    if args.workload != "c2":
        return run_layer_main(args, torch, np, ranks, hk, inputs, network, dev, world, rank, local_rank, barrier, max_over_ranks,
                              imad_peak)
    length = args.length
    cases = inputs.c2_cases(length)
    if args.cases:
        keep = set(args.cases.split(","))
        cases = [c for c in cases if "p%d_K%d_%s" % (c["p"], c["K"], "s" if c["f_signed"] else "u") in keep]
        if not cases:
            raise SystemExit("--cases matched nothing (names look like p4_K3_s)")
        cases = cases * args.case_copies      # separate buffers per copy keep a short sweep out of L2
    host_f, host_g = [], []
    for case in cases:
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"],
                                  ranks.rank_seed(case["seed"], rank))
        host_f.append(torch.from_numpy(inputs.to_storage(f)))
        host_g.append(torch.from_numpy(inputs.to_storage(g)))
    d_f = [t.to(dev) for t in host_f]
    d_g = [t.to(dev) for t in host_g]
    d_y = [torch.empty(length + c["K"] - 1, dtype=torch.int32, device=dev) for c in cases]
    macs_per_step = float(sum((length + c["K"] - 1) * c["K"] for c in cases))
    outputs_per_step = float(sum(length + c["K"] - 1 for c in cases))

    def sweep(algo):
        for c, f, g, y in zip(cases, d_f, d_g, d_y):
            hk.conv1d(f, g, c["p"], c["q"], c["f_signed"], c["g_signed"], algo=algo, out=y)

    def timed_graph(fn, steps, warmup):
        """Warm up eagerly, capture one step in a CUDA graph, replay it `steps` times between events."""
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            for _ in range(max(warmup, 3)):
                fn()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
        graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    main_algo = {"packed": hk.ALGO_PACKED32, "unpacked": hk.ALGO_UNPACKED_IMAD, "dp4a": hk.ALGO_DP4A,
                 "emu64": hk.ALGO_PACKED64EMU}[args.algo]
    total_ms = max_over_ranks(timed_graph(lambda: sweep(main_algo), args.steps, args.warmup))
    if rank == 0:
        sampler.keep_busy_until_sampled(lambda: sweep(main_algo), torch.cuda.synchronize)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = total_ms / args.steps
    value = ranks.whole_job_rate(macs_per_step, args.steps, total_ms, world)
    launches_per_step = len(cases)

    # roofline of the dominant kernel (conv1d_packed): 1 input byte + 4 output bytes per output
    avg_launch_s = total_ms * 1e-3 / (args.steps * launches_per_step)
    bytes_per_launch = 5.0 * outputs_per_step / launches_per_step
    achieved_gbs = bytes_per_launch / avg_launch_s / 1e9
    traffic = None
    rec = NCU_TRAFFIC.get("conv1d_bs")
    if args.algo == "packed" and rec and rec.get("sha256") == _source_hash("hikonv_conv1d_bs.cu") and \
            rec.get("sha256_run") == _source_hash("hikonv_conv1d_run.cuh"):
        traffic = rec["bytes_per_output"] * outputs_per_step / launches_per_step
    roofline = {"bound": "hbm", "achieved": achieved_gbs, "peak": hbm_peak_gbs, "unit": "GB/s",
                "frac": achieved_gbs / hbm_peak_gbs, "traffic": traffic, "peak_kind": "of " + peak_kind,
                "kernel": {"packed": "conv1d_bs_kernel", "unpacked": "conv1d_unpacked_tc_kernel",
                           "dp4a": "conv1d_dp4a_tc_kernel", "emu64": "conv1d_emu64_kernel"}[args.algo], "bytes_per_output": 5,
                "traffic_note": ("DRAM bytes per launch under ncu in steady state (consecutive launches over rotating buffers, "
                                 "caches not flushed between them)" if traffic is not None else
                                 "null: the kernel source has changed since the DRAM counters were taken")}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {"packed": "int64", "emu64": "int128"}.get(args.algo, "int32"), "data": "synthetic",
        "config": {"workload": "c2: 1-D bitwidth sweep, %d full convolutions of length 2^%d (p=q=1..8, K=3/5/7, unsigned+signed), "
                               "int8-stored codes in, int32 out" % (len(cases), length.bit_length() - 1),
                   "l2": "inputs larger than L2: every launch of a step has its own input and output buffers (%.1f GB per step)"
                         % ((outputs_per_step * 4 + len(cases) * length) / 1e9),
                   "launch": "one CUDA graph replay per step", "algo": args.algo},
        "gpu_launches": args.steps * launches_per_step,
        "roofline": roofline,
    }
    if clocks is not None:
        line["clocks"] = clocks

    if rank == 0 and world == 1 and not args.cases:
        # ---- end to end: pinned host buffers through the host-buffer entry point, copies inside the timed region
        # two streams, each with its own device workspace and pinned result buffer, take the cases in turn, so
        # that one case's result copy (device to host) overlaps the next case's input copy (host to device)
        streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
        wss = [torch.empty(hk.conv1d_host_workspace_bytes(length, 7), dtype=torch.uint8, device=dev) for _ in range(2)]
        pin_f = [t.pin_memory() for t in host_f]
        pin_g = [t.pin_memory() for t in host_g]
        pin_ys = [torch.empty(length + 6, dtype=torch.int32).pin_memory() for _ in range(2)]

        def e2e_step():
            for i, (c, f, g) in enumerate(zip(cases, pin_f, pin_g)):
                k = i % 2
                hk.conv1d_host(f, g, c["p"], c["q"], c["f_signed"], c["g_signed"], pin_ys[k][: length + c["K"] - 1], wss[k],
                               algo=main_algo, stream=streams[k])

        def e2e_run(steps):
            cur = torch.cuda.current_stream(dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(cur)
            for st in streams:
                st.wait_event(e0)
            for _ in range(steps):
                e2e_step()
            for st in streams:
                done = torch.cuda.Event()
                done.record(st)
                cur.wait_event(done)
            e1.record(cur)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)

        e2e_run(1)
        e2e_ms = e2e_run(args.e2e_steps) / args.e2e_steps
        line["e2e"] = {"value": macs_per_step / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(sum(t.numel() for t in host_f) + sum(t.numel() for t in host_g)),
                       "d2h_bytes_per_step": int(outputs_per_step * 4), "ms_per_step": e2e_ms}
        del pin_f, pin_ys, wss

        # ---- the comparator on the same sweep, and per-case times
        if not args.no_extra:
            extra = {}
            un_ms = timed_graph(lambda: sweep(hk.ALGO_UNPACKED_IMAD), args.steps, args.warmup) / args.steps
            extra["c2_unpacked"] = {"value": macs_per_step / (un_ms * 1e-3), "unit": UNIT, "ms_per_step": un_ms,
                                    "hbm_frac": 5.0 * outputs_per_step / (un_ms * 1e-3) / 1e9 / hbm_peak_gbs}
            del d_y
            extra["c1"] = small_case(torch, hk, inputs, dev)
            d_fd = {}
            for i, c in enumerate(cases):
                if c["p"] in (1, 2, 4):      # the widths that divide a byte have a dense-input entry point
                    vals = inputs.from_storage(host_f[i].numpy(), c["f_signed"])
                    d_fd[i] = torch.from_numpy(inputs.to_dense(vals, c["p"])).to(dev)
            extra["c2_by_bits"] = per_bitwidth_table(torch, hk, cases, d_f, d_g, length, d_fd)
            # packed against comparator per bitwidth (the six cases of a width summed); a case counts as a tie when
            # the two medians differ by no more than the larger run-to-run spread of the two
            by_width = {}
            slower, ties, faster = [], [], []
            for name, row in extra["c2_by_bits"].items():
                w = by_width.setdefault(name.split("_")[0], {"packed_us": 0.0, "unpacked_us": 0.0})
                w["packed_us"] += row["packed_us"]
                w["unpacked_us"] += row["unpacked_us"]
                spread = max(row["packed_spread_us"], row["unpacked_spread_us"])
                if abs(row["packed_us"] - row["unpacked_us"]) <= spread:
                    ties.append(name)
                elif row["packed_us"] < row["unpacked_us"]:
                    faster.append(name)
                else:
                    slower.append(name)
            for w in by_width.values():
                w["unpacked_over_packed"] = w["unpacked_us"] / w["packed_us"]
            extra["c2_packed_vs_unpacked"] = {
                "by_bitwidth": by_width, "repeats_per_cell": TABLE_REPEATS,
                "cases_packed_faster": sorted(faster), "cases_tied_within_spread": sorted(ties),
                "cases_packed_not_faster": sorted(slower)}
            del d_fd
            del d_f, d_g
            torch.cuda.empty_cache()
            extra.update(layer_workloads(torch, np, hk, inputs, network, dev, imad_peak))
            extra["peaks"] = peaks
            line["extra"] = extra
        line["cpu_baseline"] = cpu_baseline(1 << 22)

    if rank == 0:
        print(json.dumps(line), flush=True)
    ranks.shutdown()
    return 0


def run_layer_main(args, torch, np, ranks, hk, inputs, network, dev, world, rank, local_rank, barrier, max_over_ranks, imad_peak):
    """Main line for --workload c3/c4/c5: a step is one layer (or one network pass) on this rank's batch,
    timed with one event pair per step and an L2 flush (256 MB memset) before each step."""
    if args.algo not in ("packed", "unpacked"):
        raise SystemExit("--algo %s exists for the 1-D sweep only" % args.algo)
    algo = hk.ALGO_PACKED32 if args.algo == "packed" else hk.ALGO_UNPACKED_IMAD
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    launches = 0
    if args.workload in ("c3", "c4"):
        shape = dict(inputs.C3_SHAPE if args.workload == "c3" else inputs.C4_SHAPE)
        if args.batch:
            shape["B"] = args.batch
        shape["seed"] = ranks.rank_seed(shape["seed"], rank)
        x, w = inputs.layer_case(shape)
        d_x = torch.from_numpy(inputs.to_storage(x)).to(dev)
        d_w = torch.from_numpy(inputs.to_storage(w)).to(dev)
        ws = torch.empty(hk.conv2d_workspace_bytes(shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["pad"]),
                         dtype=torch.uint8, device=dev)
        rq = (shape["shift"], shape["lo"], shape["hi"]) if shape["requant"] else None
        Ho = shape["H"] + 2 * shape["pad"] - shape["K"] + 1
        Wo = shape["W"] + 2 * shape["pad"] - shape["K"] + 1
        o = torch.empty((shape["B"], shape["Co"], Ho, Wo), dtype=torch.int8 if rq else torch.int32, device=dev)
        macs = float(shape["B"]) * shape["Co"] * Ho * Wo * shape["Ci"] * shape["K"] ** 2
        muls = hk.conv2d_multiplies(shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["pad"],
                                    shape["p"], shape["q"], shape["x_signed"], shape["w_signed"], algo)

        def step():
            hk.conv2d(d_x, d_w, shape["pad"], shape["p"], shape["q"], shape["x_signed"], shape["w_signed"], requant=rq,
                      algo=algo, workspace=ws, out=o)
        launches_per_step = 2           # one packing launch, one layer launch
        name = "%s: 2-D layer %dx%dx%dx%d -> %d channels, %dx%d, pad %d, p=%d q=%d" % (
            args.workload, shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["K"], shape["pad"],
            shape["p"], shape["q"])
        h2d = d_x.numel() + d_w.numel()
        d2h = o.numel() * o.element_size()
    else:
        x, layers, head_w = inputs.c5_network(seed=ranks.rank_seed(5, rank), batch=args.batch or 64)
        d_x = torch.from_numpy(inputs.to_storage(x)).to(dev)
        net = network.CompactCnn(layers, head_w, device=dev)
        if args.c5_tiles == "tune":
            tiles = net.tune_tiles(d_x, algo=algo)          # set-up: the network times tile shapes once per input shape
        else:                                               # "auto": the library's own tiles; else tile values found earlier, one per layer
            tiles = [None] * len(layers) if args.c5_tiles == "auto" else [{"tile": int(t)} if int(t) else None for t in args.c5_tiles.split(",")]
            net.set_tiles(d_x.shape, tiles, algo=algo)
        macs, muls = 0.0, 0.0
        H, W = x.shape[2], x.shape[3]
        for L, tile in zip(layers, tiles):
            Co, Ci, K, _ = L["w"].shape
            macs += float(x.shape[0]) * Co * H * W * Ci * K * K
            muls += hk.conv2d_multiplies(x.shape[0], Ci, H, W, Co, K, L["pad"], L["p"], L["q"], L["x_signed"], L["w_signed"], algo, tile)
            if L["pool"]:
                H, W = H // 2, W // 2
        macs += float(x.shape[0]) * head_w.shape[0] * H * W * head_w.shape[1]
        muls += hk.conv2d_multiplies(x.shape[0], head_w.shape[1], H, W, head_w.shape[0], 1, 0, 4, 4, False, True, algo)

        def step():
            net.forward(d_x, algo=algo)
        launches_per_step = 2 * 9       # nine layers of two launches (packing + layer; the four pools run inside their layers)
        name = ("c5: compact 4-bit CNN, batch %d, 3x160x320, 8 conv3x3 + 4 pools + 1x1 head; tiles %s: %s"
                % (x.shape[0], {"tune": "timed once at set-up", "auto": "the library's own"}.get(args.c5_tiles, "given"),
                   [t["tile"] if t else None for t in tiles]))
        h2d = d_x.numel()
        d2h = x.shape[0] * 36 * H * W * 4

    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    barrier()
    total = 0.0
    for _ in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step()
        e1.record()
        e1.synchronize()
        total += e0.elapsed_time(e1)
    barrier()
    total = max_over_ranks(total)
    if rank == 0:
        sampler.keep_busy_until_sampled(step, torch.cuda.synchronize)
    clocks = sampler.stop() if rank == 0 else None
    ms = total / args.steps
    line = {
        "metric": METRIC, "value": ranks.whole_job_rate(macs, args.steps, total, world), "unit": UNIT, "n_gpus": world,
        "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int64" if args.algo == "packed" else "int32", "data": "synthetic",
        "config": {"workload": name, "algo": args.algo, "l2": "flushed before every step (256 MB memset outside the timed events)"},
        "gpu_launches": args.steps * launches_per_step, "clocks": clocks,
    }
    if muls is not None:
        line["roofline"] = alu_roofline(muls, ms, imad_peak, args.algo, args.workload)
        line["roofline"]["kernel"] = "conv2d_kernel" + (" (nine layer launches, multiplies summed)" if args.workload == "c5" else "")
    if rank == 0:
        print(json.dumps(line), flush=True)
    ranks.shutdown()
    return 0


def alu_roofline(muls: float, ms: float, imad_peak: dict, key: str, workload: str = None) -> dict:
    """Multiplies executed per second against the rate of that multiply: `peak` is the rate the library's own
    register-only kernel reached on this GPU (hikonv_pipe_rate) when it was measured, `frac_of_derived` divides by
    SMs x lanes per clock x maximum SM clock instead.  The step also holds the packing kernel of the layer."""
    achieved = muls / (ms * 1e-3)
    derived = imad_peak[key]
    measured = imad_peak.get(key + "_measured")
    peak = measured if measured else derived
    out = {"bound": "alu", "achieved": achieved / 1e12, "peak": peak / 1e12, "unit": "T multiply-add/s",
           "frac": achieved / peak, "traffic": None,
           "peak_kind": "of measured (register-only multiply-add kernel, this run)" if measured else "of derived",
           "frac_of_derived": achieved / derived, "derived_peak": derived / 1e12}
    # Issue model: a scheduler spends the measured cycles on every warp-wide multiply-add and on every other warp
    # instruction of the layer kernel (counted under ncu); the sum over the device's schedulers is the time the layer
    # kernel cannot go below with this instruction mix, to be read against the step (which also holds the packing launch).
    rec, issue = NCU_INSTRUCTIONS.get(workload or ""), imad_peak.get("issue")
    if key == "packed" and rec and issue and rec["sha256"] == _source_hash("hikonv_conv2d.cu"):
        mads = muls / 32.0
        others = rec["warp_instructions"] - mads
        cycles = issue["cycles_per_wide_multiply_add"] * mads + issue["cycles_added_per_other_instruction"] * others
        out["issue_model"] = {"wide_multiply_add_warp_instructions": mads, "other_warp_instructions": others,
                              "modelled_layer_kernel_ms": cycles / (issue["schedulers"] * issue["clock_hz"]) * 1e3,
                              "multiply_share_of_modelled_cycles": issue["cycles_per_wide_multiply_add"] * mads / cycles}
    return out


def small_case(torch, hk, inputs, dev):
    """C1 (4096 codes, K = 3, unsigned 4-bit): microseconds per launch inside a graph of 100 launches.  At this
    size the launch itself is the cost; the case is there for parity, not for throughput."""
    f, g = inputs.c1()
    d_f = torch.from_numpy(inputs.to_storage(f)).to(dev)
    d_g = torch.from_numpy(inputs.to_storage(g)).to(dev)
    y = torch.empty(f.size + g.size - 1, dtype=torch.int32, device=dev)
    row = {}
    for name, algo in (("packed_us", hk.ALGO_PACKED32), ("unpacked_us", hk.ALGO_UNPACKED_IMAD)):
        def fn():
            for _ in range(100):
                hk.conv1d(d_f, d_g, 4, 4, False, False, algo=algo, out=y)
        fn()
        torch.cuda.synchronize()
        g_ = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_):
            fn()
        g_.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(5):
            g_.replay()
        e1.record()
        torch.cuda.synchronize()
        row[name] = e0.elapsed_time(e1) * 1e3 / 500
    row["macs"] = float(y.numel()) * g.size
    return row


def per_bitwidth_table(torch, hk, cases, d_f, d_g, length, d_fd):
    """Microseconds per launch for every sweep case, packed, comparator and the packed method on an emulated
    64x64 multiplier (`emu64_us`), the byte dot-product comparator (`dp4a_us`), and for the 1-, 2- and 4-bit cases
    the packed kernel on dense input (8 / p codes per byte; `dense_hbm_bytes_per_output` = 4 + p / 8).  Each
    timed graph holds 12 launches that rotate over the three inputs of the same bitwidth and signedness and
    over three output buffers (240 MB per cycle), so no launch finds its data in L2.  Every cell is the median
    of TABLE_REPEATS timings of two graph replays; `*_spread_us` is their max - min."""
    table = {}
    ys = [torch.empty(length + 6, dtype=torch.int32, device=d_f[0].device) for _ in range(3)]
    for i, c in enumerate(cases):
        same = [j for j, o in enumerate(cases) if o["p"] == c["p"] and o["f_signed"] == c["f_signed"]]
        row = {}
        kinds = [("packed_us", hk.ALGO_PACKED32), ("unpacked_us", hk.ALGO_UNPACKED_IMAD), ("emu64_us", hk.ALGO_PACKED64EMU),
                 ("dp4a_us", hk.ALGO_DP4A)]
        if i in d_fd:
            kinds.append(("dense_us", None))
            row["dense_hbm_bytes_per_output"] = 4.0 + c["p"] / 8.0
        for name, algo in kinds:
            def fn():
                for r in range(12):
                    src = same[r % len(same)]
                    out = ys[r % 3][: length + c["K"] - 1]
                    if algo is None:
                        hk.conv1d_dense(d_fd[src], length, d_g[i], c["p"], c["q"], c["f_signed"], c["g_signed"], out=out)
                    else:
                        hk.conv1d(d_f[src], d_g[i], c["p"], c["q"], c["f_signed"], c["g_signed"], algo=algo, out=out)
            fn()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            g.replay()
            torch.cuda.synchronize()
            reps = []
            for _ in range(TABLE_REPEATS):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                g.replay()
                g.replay()
                e1.record()
                torch.cuda.synchronize()
                reps.append(e0.elapsed_time(e1) * 1e3 / 24)
            row[name] = statistics.median(reps)
            row[name.replace("_us", "_spread_us")] = max(reps) - min(reps)
        table["p%d_K%d_%s" % (c["p"], c["K"], "s" if c["f_signed"] else "u")] = row
    return table


def layer_workloads(torch, np, hk, inputs, network, dev, imad_peak):
    """2-D layers and the compact CNN: event-timed launches with an L2 flush before each."""
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def time_fn(fn, iters=10):
        fn()
        fn()
        torch.cuda.synchronize()
        total = 0.0
        for _ in range(iters):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
        return total / iters

    for name, shape in (("c3", inputs.C3_SHAPE), ("c4", inputs.C4_SHAPE)):
        x, w = inputs.layer_case(shape)
        d_x = torch.from_numpy(inputs.to_storage(x)).to(dev)
        d_w = torch.from_numpy(inputs.to_storage(w)).to(dev)
        ws = torch.empty(hk.conv2d_workspace_bytes(shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["pad"]),
                         dtype=torch.uint8, device=dev)
        rq = (shape["shift"], shape["lo"], shape["hi"]) if shape["requant"] else None
        Ho = shape["H"] + 2 * shape["pad"] - shape["K"] + 1
        Wo = shape["W"] + 2 * shape["pad"] - shape["K"] + 1
        o = torch.empty((shape["B"], shape["Co"], Ho, Wo), dtype=torch.int8 if rq else torch.int32, device=dev)
        macs = float(shape["B"]) * shape["Co"] * Ho * Wo * shape["Ci"] * shape["K"] ** 2
        rec = {"macs": macs}
        for key, algo in (("packed", hk.ALGO_PACKED32), ("unpacked", hk.ALGO_UNPACKED_IMAD)):
            ms = time_fn(lambda: hk.conv2d(d_x, d_w, shape["pad"], shape["p"], shape["q"], shape["x_signed"], shape["w_signed"],
                                           requant=rq, algo=algo, workspace=ws, out=o))
            muls = hk.conv2d_multiplies(shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["pad"],
                                        shape["p"], shape["q"], shape["x_signed"], shape["w_signed"], algo)
            rec[key] = {"ms": ms, "value": macs / (ms * 1e-3), "unit": UNIT, "roofline": alu_roofline(muls, ms, imad_peak, key, name)}
        rec["layout"] = hk.conv2d_layout(shape["B"], shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["pad"],
                                         shape["p"], shape["q"], shape["x_signed"], shape["w_signed"])
        rec["packed_over_unpacked"] = rec["unpacked"]["ms"] / rec["packed"]["ms"]
        if rq and shape["p"] == 4 and shape["q"] == 4:
            # the same layer with all three tensors stored densely (two 4-bit codes per byte): half the bytes per tensor
            dx = torch.from_numpy(inputs.to_dense(x, 4)).to(dev)
            dw = torch.from_numpy(inputs.to_dense(w, 4)).to(dev)
            do = torch.empty(o.numel() // 2, dtype=torch.uint8, device=dev)
            ms = time_fn(lambda: hk.conv2d_dense(dx, x.shape, 4, dw, w.shape, 4, shape["pad"], 4, 4, shape["x_signed"], shape["w_signed"],
                                                 requant=rq, out_store_bits=4, workspace=ws, out=do))
            n_out = float(o.numel())
            rec["dense"] = {"ms": ms, "value": macs / (ms * 1e-3), "unit": UNIT,
                            "hbm_bytes_per_output": (dx.numel() + dw.numel() + do.numel()) / n_out,
                            "byte_storage_hbm_bytes_per_output": (d_x.numel() + d_w.numel() + o.numel()) / n_out}
            del dx, dw, do
        out[name] = rec
        del d_x, d_w, o

    # the C3 layer shape at every bitwidth p = q = 1 .. 8 (signed codes, exact int32 sums): packed against one product per multiply
    by_bits = {}
    B, Ci, H, W, Co = 32, 64, 56, 56, 64
    for p in range(1, 9):
        x, w = inputs.conv2d_case(B, Ci, H, W, Co, 3, p, p, True, True, seed=40 + p)
        d_x = torch.from_numpy(inputs.to_storage(x)).to(dev)
        d_w = torch.from_numpy(inputs.to_storage(w)).to(dev)
        ws = torch.empty(hk.conv2d_workspace_bytes(B, Ci, H, W, Co, 3, 1), dtype=torch.uint8, device=dev)
        o = torch.empty((B, Co, H, W), dtype=torch.int32, device=dev)
        row = {}
        for key, algo in (("packed", hk.ALGO_PACKED32), ("unpacked", hk.ALGO_UNPACKED_IMAD)):
            row[key + "_ms"] = time_fn(lambda: hk.conv2d(d_x, d_w, 1, p, p, True, True, algo=algo, workspace=ws, out=o), iters=5)
        L = hk.conv2d_layout(B, Ci, H, W, Co, 3, 1, p, p, True, True)
        row["unpacked_over_packed"] = row["unpacked_ms"] / row["packed_ms"]
        row["layout"] = {k: L[k] for k in ("N", "S", "J", "M")}
        by_bits["p%d" % p] = row
        del d_x, d_w, o, ws
    out["c3_shape_by_bitwidth"] = by_bits

    x, layers, head_w = inputs.c5_network()
    d_x = torch.from_numpy(inputs.to_storage(x)).to(dev)
    net = network.CompactCnn(layers, head_w, device=dev)
    macs = 0.0
    H, W = x.shape[2], x.shape[3]
    for L in layers:
        Co, Ci, K, _ = L["w"].shape
        macs += float(x.shape[0]) * Co * H * W * Ci * K * K
        if L["pool"]:
            H, W = H // 2, W // 2
    macs += float(x.shape[0]) * head_w.shape[0] * H * W * head_w.shape[1]
    rec = {"macs": macs}
    for key, algo in (("packed", hk.ALGO_PACKED32), ("unpacked", hk.ALGO_UNPACKED_IMAD)):
        untuned_ms = time_fn(lambda: net.forward(d_x, algo=algo), iters=5)
        tiles = net.tune_tiles(d_x, algo=algo)              # set-up: the network times tile shapes once per input shape
        ms = time_fn(lambda: net.forward(d_x, algo=algo), iters=5)
        # multiplies the nine layer launches execute (positions incl. halo x Co x Ci x K x J, summed)
        muls, Hl, Wl = 0.0, x.shape[2], x.shape[3]
        for L, tile in zip(layers, tiles):
            Co, Ci, K, _ = L["w"].shape
            muls += hk.conv2d_multiplies(x.shape[0], Ci, Hl, Wl, Co, K, L["pad"], L["p"], L["q"], L["x_signed"], L["w_signed"], algo, tile)
            if L["pool"]:
                Hl, Wl = Hl // 2, Wl // 2
        muls += hk.conv2d_multiplies(x.shape[0], head_w.shape[1], Hl, Wl, head_w.shape[0], 1, 0, 4, 4, False, True, algo)
        rec[key] = {"ms": ms, "value": macs / (ms * 1e-3), "unit": UNIT, "roofline": alu_roofline(muls, ms, imad_peak, key),
                    "ms_with_the_library_s_own_tiles": untuned_ms, "tuned_tiles": [t["tile"] if t else None for t in tiles]}
    rec["packed_over_unpacked"] = rec["unpacked"]["ms"] / rec["packed"]["ms"]
    out["c5"] = rec
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the comparator, per-case and 2-D workloads")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--length", type=int, default=1 << 24, help="signal length of the sweep (benchmark value: 2^24)")
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "c5"],
                    help="c2 = 1-D sweep (default, the benchmark step); c3/c4 = one 2-D layer; c5 = the compact CNN")
    ap.add_argument("--c5-tiles", default="tune",
                    help="c5 only: tune = time tile shapes once at set-up (default); auto = the library's own tiles; or the tile "
                         "values of an earlier tuning pass, one per conv3x3 layer, comma-separated, 0 = automatic (for profiling)")
    ap.add_argument("--cases", default="", help="c2 only: comma-separated subset such as p4_K3_s,p8_K7_u (for profiling)")
    ap.add_argument("--case-copies", type=int, default=3, help="with --cases: buffer copies per case")
    ap.add_argument("--batch", type=int, default=0, help="c3/c4/c5: override the batch size (for profiling)")
    ap.add_argument("--algo", default="packed", choices=["packed", "unpacked", "dp4a", "emu64"],
                    help="which kernel the main line times (dp4a and emu64: the 1-D sweep only)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
