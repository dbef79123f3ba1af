#!/usr/bin/env python
"""Benchmark of the BitLinear W1.58A8 hot path on B200.

Headline (the line's `value`): packed-weight GB/s of the M=1 streaming kernel over a whole ~2B-parameter
backbone - one step = the sweep over 30 blocks x {qkv, out, gate/up, down} = 120 independent GEMVs streaming
521 MB of packed ternary weights (4x the 126 MB L2, so all weights are read cold), issued as one grouped launch.
Secondary figures in the same JSON line (`extra`): the same matrices as a chain of single launches, M=8, the
M=4096 tcgen05 GEMM (int8 TOPS), the 30-block encoder forward (states/s); plus the CPU oracle timed on the host
cores and the roofline fraction of the dominant kernel.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--layers L] [--sections ...]

Under torchrun (N > 1) every rank runs the same step on its own replica of the weights and its own states
(no collective on the data path); rank 0 prints the aggregate.
"""
from __future__ import annotations

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

import torch  # noqa: E402

from paper_2604_24273_b200 import inputs  # noqa: E402

METRIC = "BitLinear GB/s (M=1) and int8 TOPS (M=4096) on 1 B200 as % of roofline"
BLOCK = [("qkv", 2560, 3840), ("out", 2560, 2560), ("gateup", 2560, 13824), ("down", 6912, 2560)]  # (name, K, N)
FULL_LAYERS = 30
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
INT8_OVER_BF16 = 2.0  # nominal dense int8 : bf16 tensor throughput on B200 (4.5 : 2.25 PFLOP/s)
# DRAM bytes (read + write) of one gemv_multi_dp4a_kernel<1> launch per backbone block, from an ncu capture of the
# 8-block case (dram__bytes_read.sum 138.987 MB + dram__bytes_write.sum 3.904 MB, means of two launches of the kernel as
# it is now); every weight byte is read exactly once, so traffic scales with the number of blocks.  Set to None whenever
# that kernel changes.
HEADLINE_TRAFFIC_PER_BLOCK = (138.987008e6 + 3.904e6) / 8


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def packed_bytes_per_layer():
    return sum(k * n // 4 for _, k, n in BLOCK)


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except ValueError:
                continue
            for nme, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------- helpers
def dist_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def barrier_sync(world):
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
        torch.cuda.synchronize()


def max_over_ranks(ms: float, world: int) -> float:
    if world == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device="cuda")
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def time_graph(graph, steps, warmup, world):
    """W warm-up replays, then K timed replays between CUDA events on the launching stream; max over ranks (ms)."""
    for _ in range(warmup):
        graph.replay()
    barrier_sync(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    barrier_sync(world)
    return max_over_ranks(e0.elapsed_time(e1), world)


def time_rounds(graph, steps, rounds=10):
    """`rounds` further passes of `steps` replays each (this rank only): the spread of the per-step time in ms."""
    per = []
    for _ in range(rounds):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        per.append(e0.elapsed_time(e1) / steps)
    return {"rounds": rounds, "steps_per_round": steps, "median": statistics.median(per), "min": min(per), "max": max(per)}


def capture(fn):
    """Runs fn once eagerly, then captures it into a CUDA graph (the library launches on the current stream).
    Returns (graph, number of library kernel launches inside the graph)."""
    from paper_2604_24273_b200 import bitrl

    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    n0 = bitrl.launch_count()
    with torch.cuda.graph(g):
        fn()
    launches = bitrl.launch_count() - n0
    torch.cuda.synchronize()
    return g, launches


def gemm_kernel_name(bitrl, M, K, N):
    """The form of the tensor-core kernel the launcher takes for this shape, as the library reports it."""
    tok, splits, kind = bitrl.gemm_plan(M, K, N)
    form = {bitrl.GEMM_SINGLE: "single CTAs", bitrl.GEMM_SPLIT_SCRATCH: f"split-K x{splits} through scratch",
            bitrl.GEMM_SPLIT_CLUSTER: f"split-K x{splits} inside a cluster", bitrl.GEMM_PAIRED: "CTA pairs (cta_group::2)"}[kind]
    return f"gemm_i8_kernel<TOK={tok}>, {form}"


def build_backbone(bitrl, n_layers, seed=5000):
    """Blocks of ternary weights.  Master weights are drawn on the GPU (N(0, 0.02), seeded per matrix) to keep
    set-up short, packed by the library and dropped; only the packed handles stay (17.4 MB per block)."""
    layers = []
    gen = torch.Generator(device="cuda")
    for l in range(n_layers):
        blk = []
        for j, (_, k, n) in enumerate(BLOCK):
            gen.manual_seed(seed + 4 * l + j)
            W = torch.randn(n, k, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W
            blk.append(bitrl.Linear.from_master(W))
            del W
        layers.append(tuple(blk))
    torch.cuda.synchronize()
    return layers


# ------------------------------------------------------------------------------------------ oracle legs
def oracle_block0():
    import oracle

    mats = []
    for j, (_, k, n) in enumerate(BLOCK):
        W = inputs.master_weights(n, k, 5000 + j)
        Wq, g = oracle.ternarize(W.numpy())
        mats.append((Wq, g, inputs.bf16_bits(inputs.activations(1, k, 2001))))

    def step():
        for Wq, g, x in mats:
            oracle.bitlinear(x, Wq, g)
    return step


def oracle_decode_sample(min_seconds=10.0):
    """The CPU oracle, as it stands, on the M=1 decode workload: block 0's four matrices (69.5 M weights,
    17.4 MB packed), quant -> contract -> rescale, repeated for about `min_seconds` of CPU work."""
    step = oracle_block0()
    nbytes = packed_bytes_per_layer()
    reps, t0 = 0, time.perf_counter()
    while True:
        step()
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return {"value": reps * nbytes / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"block 0 (qkv, out, gate/up, down; 17.4 MB packed) at M=1, {reps} passes in {dt:.1f} s; the "
                      "oracle threads over token rows, so M=1 runs on one core"}


def oracle_batched_samples():
    """The oracle beside the other half of the metric: a sample of token rows of both M = 4096 shapes (quant ->
    contract -> rescale) and one encoder block on one 32-token state, each with one thread and with every core this
    process may run on."""
    import oracle

    cores = oracle.default_threads()
    out = {"kind": "oracle", "cores_all": cores}
    for K, N, seed in ((2560, 6912, 1005), (6912, 2560, 1004)):
        Wq, g = oracle.ternarize(inputs.master_weights(N, K, seed).numpy())
        for label, threads, rows in (("1_thread", 1, 128), ("all_cores", cores, min(4096, 64 * cores))):
            x = inputs.bf16_bits(inputs.activations(rows, K, 2400))
            t0 = time.perf_counter()
            oracle.bitlinear(x, Wq, g, threads=threads)
            dt = time.perf_counter() - t0
            out[f"m4096_k{K}_n{N}_{label}"] = {
                "TOPS": 2.0 * rows * N * K / dt / 1e12, "cores": threads, "seconds": dt,
                "sample": f"{rows} of the 4096 token rows"}
    layer = [oracle.ternarize(w.numpy()) for w in inputs.encoder_layer_weights(0)]
    h = inputs.bf16_bits(inputs.activations(32, 2560, 6002))
    for label, threads in (("1_thread", 1), ("all_cores", cores)):
        t0 = time.perf_counter()
        oracle.encoder_block(h, 6912, 20, 5, layer, threads=threads)
        dt = time.perf_counter() - t0
        out[f"encoder_block_1_state_x32_tokens_{label}"] = {
            "states_per_s_30_blocks": 1.0 / (dt * 30), "cores": threads, "seconds_per_block": dt,
            "sample": "block 0 on one 32-token state (identity attention); a full forward is 30 such blocks"}
    return out


def run_reference(args):
    """--impl reference: the CPU oracle on the same metric/config, each step a bounded sample."""
    rank, _, _ = dist_env()
    if rank != 0:
        return
    step = oracle_block0()
    nbytes = packed_bytes_per_layer()
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    gbs = args.steps * nbytes / dt / 1e9
    sample = "each step = block 0 of the backbone (4 matrices, 17.4 MB packed) at M=1 on one host core"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 x ternary(2-bit) -> int32", "data": "synthetic",
        "config": {"workload": "configs[1]: decode GEMV sweep, M=1, shapes of a ~2B BitNet b1.58 block",
                   "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------ ours
def run_ours(args):
    from paper_2604_24273_b200 import bitrl

    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local))
    bitrl.lib()
    peaks, peak_src = load_peaks()
    dev = torch.device("cuda", local)
    n_layers = args.layers
    sections = set(s for s in args.sections.split(",") if s)
    sub_steps = max(3, args.steps // 4)

    layers = build_backbone(bitrl, n_layers)
    bytes_step = n_layers * packed_bytes_per_layer()

    # ---------------- headline: the M = 1 sweep over every matrix of the backbone.  The 4 * n_layers GEMVs are
    # independent (same activations, distinct weights), so they go through the grouped entry point: one launch of
    # one persistent kernel per step.
    def decode_setup(M):
        # the two activation tensors share one device buffer, and so do the outputs of each block: a step's inputs and
        # its result then cross PCIe as one copy each way in the end-to-end measurement
        xflat = torch.empty((M * (2560 + 6912),), dtype=torch.bfloat16, device=dev)
        xs = {2560: xflat[:M * 2560].view(M, 2560), 6912: xflat[M * 2560:].view(M, 6912)}
        for k in xs:
            xs[k].copy_(inputs.activations(M, k, 2000 + M))
        per_block = M * sum(n for _, _, n in BLOCK)
        yall = torch.empty((n_layers * per_block,), dtype=torch.bfloat16, device=dev)  # every output of a step
        ys = []
        for l in range(n_layers):
            off, row = l * per_block, []
            for _, _, n in BLOCK:
                row.append(yall[off:off + M * n].view(M, n))
                off += M * n
            ys.append(row)
        ws = [layers[l][j] for l in range(n_layers) for j in range(len(BLOCK))]
        xl = [xs[k] for _ in range(n_layers) for _, k, _ in BLOCK]
        yl = [ys[l][j] for l in range(n_layers) for j in range(len(BLOCK))]
        calls = [bitrl.MultiCall(ws[i:i + 128], xl[i:i + 128], yl[i:i + 128], bitrl.OUT_BF16)
                 for i in range(0, len(ws), 128)]

        def sweep():
            for c in calls:
                c.run()

        def chain():  # the same matrices as one launch each, in stream order (programmatic dependent launch)
            for l in range(n_layers):
                for j, (_, k, n) in enumerate(BLOCK):
                    bitrl.bitlinear_forward(layers[l][j], xs[k], bitrl.OUT_BF16, y=ys[l][j])
        xs["flat"] = xflat
        xs["yall"] = yall
        return xs, ys, sweep, chain

    xs1, ys1, step1, chain1 = decode_setup(1)
    g1, launches1 = capture(step1)  # one step

    def k_steps():
        for _ in range(args.steps):
            step1()

    # The timed region is ONE graph that holds the K steps back to back: consecutive launches are joined by programmatic
    # dependent launch, so a step's CTAs are queued (and its weight stream starts) while the previous step's last CTAs
    # drain, as in any loop that issues steps ahead of their completion.  The one-graph-per-step figure is kept beside it.
    gk, launches_k = capture(k_steps)
    sampler = ClockSampler(local).start() if rank == 0 else None
    for _ in range(args.warmup):
        g1.replay()
    gk.replay()  # the first launch of an instantiated graph also uploads it: not part of the timed region
    ms1 = time_graph(gk, 1, 0, world)
    gbs1 = world * bytes_step * args.steps / (ms1 * 1e-3) / 1e9
    us_per_launch = ms1 * 1e3 / launches_k
    spread1 = time_rounds(gk, 1)
    for key in ("median", "min", "max"):
        spread1[key] /= args.steps
    spread1["steps_per_round"] = args.steps
    ms1_single = time_graph(g1, args.steps, args.warmup, world)
    del gk

    # end to end: pinned host x -> device, the sweep, ALL of the step's outputs (4 per block, one contiguous buffer) back
    # to pinned host memory.  The two copies are nodes of the same CUDA graph as the kernel, so a step is one graph launch
    # plus the wait for its result.
    host_x = torch.cat([inputs.activations(1, k, 2001).reshape(-1) for k in (2560, 6912)]).pin_memory()
    host_y = torch.empty_like(xs1["yall"], device="cpu").pin_memory()
    h2d = host_x.numel() * 2
    d2h = host_y.numel() * 2

    def e2e_body():
        xs1["flat"].copy_(host_x, non_blocking=True)
        step1()
        host_y.copy_(xs1["yall"], non_blocking=True)

    ge, _ = capture(e2e_body)

    def e2e_step():
        ge.replay()
        torch.cuda.current_stream().synchronize()

    for _ in range(args.warmup):
        e2e_step()
    barrier_sync(world)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3, world)
    e2e_gbs = world * bytes_step * args.steps / (e2e_ms * 1e-3) / 1e9

    # The same steps two deep: a second set of device and pinned host buffers on a second stream, so that the copies
    # of one step run beside the kernel of the next (every step still copies its inputs in and all its outputs out
    # inside the timed region; the host waits for a slot's previous result before it reuses the slot).
    xs1b, _, step1b, _ = decode_setup(1)
    host_yb = torch.empty_like(host_y).pin_memory()
    slots = []
    for xs_, step_, hy_ in ((xs1, step1, host_y), (xs1b, step1b, host_yb)):
        st_ = torch.cuda.Stream()
        with torch.cuda.stream(st_):
            def body(xs_=xs_, step_=step_, hy_=hy_):
                xs_["flat"].copy_(host_x, non_blocking=True)
                step_()
                hy_.copy_(xs_["yall"], non_blocking=True)
            g_, _ = capture(body)
        slots.append((st_, g_))

    def pipelined(n):
        for i in range(n):
            st_, g_ = slots[i & 1]
            st_.synchronize()  # the slot's previous result has arrived
            with torch.cuda.stream(st_):
                g_.replay()
        for st_, _ in slots:
            st_.synchronize()

    pipelined(args.warmup)
    barrier_sync(world)
    t0 = time.perf_counter()
    pipelined(args.steps)
    e2e_pipe_ms = max_over_ranks((time.perf_counter() - t0) * 1e3, world)
    e2e_pipe_gbs = world * bytes_step * args.steps / (e2e_pipe_ms * 1e-3) / 1e9
    del slots
    clocks = sampler.stop() if sampler else None
    sampler2 = ClockSampler(local).start() if rank == 0 else None  # clocks during the secondary sections

    extra, cpu = {}, None
    gemm_roofline = []  # the int8-TOPS half of the metric: one entry per judged M = 4096 shape
    per_call_m1 = None
    if rank == 0 and "decode8" in sections:
        gc, lc = capture(chain1)
        msc = time_graph(gc, args.steps, args.warmup, 1)
        gbc = bytes_step * args.steps / (msc * 1e-3) / 1e9
        extra["chain_m1_one_launch_per_matrix"] = {"GBps": gbc, "us_per_launch": msc * 1e3 / (args.steps * lc),
                                                  "frac_of_hbm_peak": gbc / peaks["hbm_gbs"], "launches": lc}
        per_call_m1 = {"call": "bitrl_bitlinear_forward, one launch per matrix in stream order", "kernel": "gemv_kernel<1>",
                       "achieved": gbc, "unit": "GB/s", "frac": gbc / peaks["hbm_gbs"],
                       "us_per_launch": msc * 1e3 / (args.steps * lc)}
        del gc
        _, _, step8, chain8 = decode_setup(8)
        for label, fn in (("sweep_m8_grouped", step8), ("chain_m8_one_call_per_matrix", chain8)):
            g8, l8 = capture(fn)
            ms8 = time_graph(g8, args.steps, args.warmup, 1)
            gb8 = bytes_step * args.steps / (ms8 * 1e-3) / 1e9
            extra[label] = {"GBps": gb8, "ms_per_step": ms8 / args.steps, "frac_of_hbm_peak": gb8 / peaks["hbm_gbs"],
                            "launches": l8}
            del g8
            if fn is step8:  # and, as in the headline, the K steps back to back in one graph
                def k_steps8():
                    for _ in range(args.steps):
                        step8()
                g8k, _ = capture(k_steps8)
                g8k.replay()
                ms8k = time_graph(g8k, 1, 0, 1)
                gb8k = bytes_step * args.steps / (ms8k * 1e-3) / 1e9
                extra[label]["steps_in_one_graph"] = {"GBps": gb8k, "ms_per_step": ms8k / args.steps,
                                                      "frac_of_hbm_peak": gb8k / peaks["hbm_gbs"]}
                del g8k

    if rank == 0 and "pack" in sections:
        # a0, the offline step: absmean scale + ternarize + pack of the block's largest matrix (fp32 master weights, 141.6 MB;
        # three matrices in turn so that nothing is left in L2).  Algorithmic bytes: W read once, packed codes written.
        Np, Kp = 13824, 2560
        gen0 = torch.Generator(device="cuda")
        gen0.manual_seed(4242)
        Wm = [torch.randn(Np, Kp, generator=gen0, device="cuda", dtype=torch.float32) * inputs.SIGMA_W for _ in range(3)]
        pk = torch.empty((Np, Kp // 4), dtype=torch.uint8, device=dev)
        gm = torch.empty((1,), dtype=torch.float32, device=dev)

        def pack3():
            for W_ in Wm:
                bitrl.pack_ternary_static(W_, pk, gm)

        gp, lp = capture(pack3)
        usp = time_graph(gp, sub_steps, args.warmup, 1) * 1e3 / (sub_steps * 3)
        alg = Np * Kp * 4.25
        extra["pack_ternary_13824x2560"] = {"us": usp, "GBps_algorithmic": alg / (usp * 1e-6) / 1e9,
                                            "frac_of_hbm_peak": alg / (usp * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                            "passes_over_W": 2, "launches": lp / 3}
        del gp, Wm, pk, gm

    if rank == 0 and "pack5" in sections:
        # the same M = 1 sweep on the five-weights-per-byte format (1.6 bits per weight, lookup-table decode): judged on
        # microseconds per sweep against the 2-bit kernel's, and on GB/s of its own (smaller) packed bytes
        gen5 = torch.Generator(device="cuda")
        lin5 = []
        for l in range(n_layers):
            for j, (_, k, n) in enumerate(BLOCK):
                gen5.manual_seed(5000 + 4 * l + j)
                lin5.append(bitrl.Linear5.from_master(torch.randn(n, k, generator=gen5, device="cuda") * inputs.SIGMA_W))
        x5 = [xs1[k] for _ in range(n_layers) for _, k, _ in BLOCK]
        y5 = [torch.empty_like(ys1[l][j]) for l in range(n_layers) for j in range(len(BLOCK))]
        call5 = bitrl.MultiCall5(lin5, x5, y5, bitrl.OUT_BF16)
        g5, l5 = capture(call5.run)
        ms5 = time_graph(g5, args.steps, args.warmup, 1) / args.steps
        step1()
        torch.cuda.synchronize()
        same = all(torch.equal(a_, ys1[l][j]) for a_, (l, j) in zip(y5, [(l, j) for l in range(n_layers) for j in range(len(BLOCK))]))
        bytes5 = sum(w.nbytes for w in lin5)
        extra["sweep_m1_five_weights_per_byte"] = {
            "us_per_sweep": ms5 * 1e3, "us_per_sweep_2bit": ms1_single / args.steps * 1e3, "packed_bytes": bytes5,
            "GBps_of_its_own_bytes": bytes5 / (ms5 * 1e-3) / 1e9, "frac_of_hbm_peak": bytes5 / (ms5 * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "bits_per_weight": 8.0 * bytes5 / (n_layers * sum(k * n for _, k, n in BLOCK)),
            "outputs_equal_2bit_path": bool(same), "launches": l5}
        del g5, lin5, y5

    if rank == 0 and "gemm" in sections:
        # M = 4096 GEMM, both judged shapes; weights rotate over several matrices, inputs over four buffers
        i8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
        M = 4096
        gen = torch.Generator(device="cuda")
        up_only = []  # eight 2560 -> 6912 matrices (the block itself only has the fused 2560 -> 13824 one)
        for i in range(8):
            gen.manual_seed(1005 + 100 * i)
            up_only.append(bitrl.Linear.from_master(
                torch.randn(6912, 2560, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W))
        for name, K, N in (("gemm_m4096_k2560_n6912", 2560, 6912), ("gemm_m4096_k6912_n2560", 6912, 2560)):
            mats = up_only if N == 6912 else [layers[l][3] for l in range(n_layers)]
            xs = [inputs.activations(M, K, 2400 + i).to(dev) for i in range(4)]
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = torch.empty((bitrl.workspace_bytes(M, K, N),), dtype=torch.uint8, device=dev)
            q = [bitrl.quant_act(x) for x in xs]
            reps = 12

            def full():
                for i in range(reps):
                    bitrl.bitlinear_forward(mats[i % len(mats)], xs[i % 4], bitrl.OUT_BF16, y=y, workspace=ws)

            def kernel_only():
                for i in range(reps):
                    bitrl.bitlinear_forward_q(mats[i % len(mats)], *q[i % 4], bitrl.OUT_BF16, y=y)

            ops = 2.0 * M * N * K * reps
            res = {}
            for label, fn in (("layer", full), ("gemm_kernel", kernel_only)):
                g, _ = capture(fn)
                ms = time_graph(g, sub_steps, args.warmup, 1)
                tops = ops * sub_steps / (ms * 1e-3) / 1e12
                res[label] = {"TOPS": tops, "us": ms * 1e3 / (sub_steps * reps), "frac_of_int8_peak": tops / i8_peak,
                              "frac_of_nominal_4500": tops / 4500.0}
                del g
            res["int8_peak"] = f"{i8_peak:.0f} TOPS = 2 x bf16 burst peak (of {peak_src})"
            extra[name] = res
            gemm_roofline.append({
                "shape": f"M=4096 K={K} N={N}", "bound": "tensor", "unit": "TOPS", "peak": i8_peak,
                "peak_source": f"2 x bf16 burst, of {peak_src}",
                "kernel": gemm_kernel_name(bitrl, M, K, N),
                "us": res["gemm_kernel"]["us"], "achieved": res["gemm_kernel"]["TOPS"],
                "frac": res["gemm_kernel"]["frac_of_int8_peak"], "frac_of_nominal_4500": res["gemm_kernel"]["frac_of_nominal_4500"],
                "layer_us": res["layer"]["us"], "layer_achieved": res["layer"]["TOPS"],
                "layer_frac": res["layer"]["frac_of_int8_peak"],
                "layer_frac_of_nominal_4500": res["layer"]["frac_of_nominal_4500"],
                "algorithmic_ops_per_launch": 2.0 * M * N * K})
            del xs, y, ws, q

        if "critic" in sections:  # Table IV's higher-precision critic layers (W8A8, W4A8)
            # the higher-precision critic's W8A8 layer at the same M = 4096 shapes (int8 weights, nothing to decode)
            for name, K, N in (("w8a8_m4096_k2560_n6912", 2560, 6912), ("w8a8_m4096_k6912_n2560", 6912, 2560)):
                w8 = []
                for i in range(4):
                    gen.manual_seed(1400 + i)
                    w8.append(bitrl.w8_quantize(torch.randn(N, K, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W))
                xs = [inputs.activations(M, K, 2400 + i).to(dev) for i in range(4)]
                y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                ws = torch.empty((int(bitrl.lib().bitrl_w8a8_workspace_bytes(M, K)),), dtype=torch.uint8, device=dev)
                reps = 12

                def w8_layer():
                    for i in range(reps):
                        bitrl.w8a8_forward(*w8[i % 4], xs[i % 4], bitrl.OUT_BF16, y=y, workspace=ws)

                g, _ = capture(w8_layer)
                ms = time_graph(g, sub_steps, args.warmup, 1)
                tops = 2.0 * M * N * K * reps * sub_steps / (ms * 1e-3) / 1e12
                extra[name] = {"layer": {"TOPS": tops, "us": ms * 1e3 / (sub_steps * reps), "frac_of_int8_peak": tops / i8_peak,
                                         "frac_of_nominal_4500": tops / 4500.0}}
                del g, xs, y, ws, w8

            # ... and its streaming kernel at M = 1 and 8 over eight 2560 -> 13824 matrices (283 MB of int8 weights, > L2)
            w8 = []
            for i in range(8):
                gen.manual_seed(1500 + i)
                w8.append(bitrl.w8_quantize(torch.randn(13824, 2560, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W))
            for Ms in (1, 8):
                xd = inputs.activations(Ms, 2560, 2000 + Ms).to(dev)
                yd = torch.empty((Ms, 13824), dtype=torch.bfloat16, device=dev)

                def w8_sweep():
                    for wq8, sc8 in w8:
                        bitrl.w8a8_forward(wq8, sc8, xd, bitrl.OUT_BF16, y=yd)

                g, lc = capture(w8_sweep)
                ms = time_graph(g, sub_steps, args.warmup, 1) / sub_steps
                gbs = 8 * 13824 * 2560 / (ms * 1e-3) / 1e9
                extra[f"w8a8_m{Ms}_sweep_8x_k2560_n13824"] = {"GBps_of_weight_bytes": gbs, "us_per_matrix": ms * 1e3 / 8,
                                                             "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "launches": lc}
                del g
            # ... and the M = 1 sweep over the same eight matrices as ONE grouped launch
            xd = inputs.activations(1, 2560, 2001).to(dev)
            yds = [torch.empty((1, 13824), dtype=torch.bfloat16, device=dev) for _ in w8]
            call8 = bitrl.W8MultiCall(w8, [xd] * len(w8), yds, bitrl.OUT_BF16)
            g, lc = capture(call8.run)
            ms = time_graph(g, sub_steps, args.warmup, 1) / sub_steps
            gbs = 8 * 13824 * 2560 / (ms * 1e-3) / 1e9
            extra["w8a8_m1_sweep_8x_k2560_n13824_grouped"] = {"GBps_of_weight_bytes": gbs, "us_per_matrix": ms * 1e3 / 8,
                                                             "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "launches": lc}
            del g, call8, yds
            del w8

            # the INT4 critic's W4A8 layer: streaming kernel at M = 1 over eight 2560 -> 13824 matrices (141 MB packed),
            # and the whole layer at M = 4096 (int8 expansion into the workspace, then the W8A8 GEMM)
            w4 = []
            for i in range(8):
                gen.manual_seed(1600 + i)
                w4.append(bitrl.w4_quantize(torch.randn(13824, 2560, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W))
            xd = inputs.activations(1, 2560, 2001).to(dev)
            yd = torch.empty((1, 13824), dtype=torch.bfloat16, device=dev)

            def w4_sweep():
                for p4, sc4 in w4:
                    bitrl.w4a8_forward(p4, sc4, xd, bitrl.OUT_BF16, y=yd)

            g, lc = capture(w4_sweep)
            ms = time_graph(g, sub_steps, args.warmup, 1) / sub_steps
            gbs = 8 * 13824 * 2560 / 2 / (ms * 1e-3) / 1e9
            extra["w4a8_m1_sweep_8x_k2560_n13824"] = {"GBps_of_packed_bytes": gbs, "us_per_matrix": ms * 1e3 / 8,
                                                       "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "launches": lc}
            del g
            yds = [torch.empty((1, 13824), dtype=torch.bfloat16, device=dev) for _ in w4]
            call4 = bitrl.W8MultiCall(w4, [xd] * len(w4), yds, bitrl.OUT_BF16, int4=True)
            g, lc = capture(call4.run)
            ms = time_graph(g, sub_steps, args.warmup, 1) / sub_steps
            gbs = 8 * 13824 * 2560 / 2 / (ms * 1e-3) / 1e9
            extra["w4a8_m1_sweep_8x_k2560_n13824_grouped"] = {"GBps_of_packed_bytes": gbs, "us_per_matrix": ms * 1e3 / 8,
                                                               "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "launches": lc}
            del g, call4, yds, w4
            gen.manual_seed(1700)
            p4, sc4 = bitrl.w4_quantize(torch.randn(6912, 2560, generator=gen, device="cuda", dtype=torch.float32) * inputs.SIGMA_W)
            xs = [inputs.activations(M, 2560, 2400 + i).to(dev) for i in range(4)]
            y = torch.empty((M, 6912), dtype=torch.bfloat16, device=dev)
            ws = torch.empty((int(bitrl.lib().bitrl_w4a8_workspace_bytes(M, 2560, 6912)),), dtype=torch.uint8, device=dev)

            def w4_layer():
                for i in range(12):
                    bitrl.w4a8_forward(p4, sc4, xs[i % 4], bitrl.OUT_BF16, y=y, workspace=ws)

            g, _ = capture(w4_layer)
            ms = time_graph(g, sub_steps, args.warmup, 1)
            tops = 2.0 * M * 6912 * 2560 * 12 * sub_steps / (ms * 1e-3) / 1e12
            extra["w4a8_m4096_k2560_n6912"] = {"layer": {"TOPS": tops, "us": ms * 1e3 / (sub_steps * 12),
                                                         "frac_of_int8_peak": tops / i8_peak}}
            del g, xs, y, ws

        # configs[2]: batched state encoding, M = 64 and 256 (one token per state), the whole layer per call
        for M in (64, 256):
            for K, N in ((2560, 6912), (6912, 2560)):
                mats = up_only if N == 6912 else [layers[l][3] for l in range(n_layers)]
                xs = [inputs.activations(M, K, 2500 + i).to(dev) for i in range(4)]
                y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                ws = torch.empty((bitrl.workspace_bytes(M, K, N),), dtype=torch.uint8, device=dev)
                reps = 24

                def small():
                    for i in range(reps):
                        bitrl.bitlinear_forward(mats[i % len(mats)], xs[i % 4], bitrl.OUT_BF16, y=y, workspace=ws)

                g, lc = capture(small)
                ms = time_graph(g, sub_steps, args.warmup, 1)
                us = ms * 1e3 / (sub_steps * reps)
                extra[f"layer_m{M}_k{K}_n{N}"] = {"us": us, "TOPS": 2.0 * M * N * K / (us * 1e-6) / 1e12,
                                                  "kernel": gemm_kernel_name(bitrl, M, K, N),
                                                  "packed_GBps": N * K / 4 / (us * 1e-6) / 1e9,
                                                  "launches_per_layer": lc / reps}
                del g, xs, y, ws

    if world > 1 and "encoder" in sections:
        # config 5 with its 4096 token rows sharded over the ranks (strong scaling: the same 128 states, fewer per GPU);
        # rows are independent, so every rank encodes its own contiguous block of states and nothing is exchanged
        from paper_2604_24273_b200.sharding import shard_rows

        row0, rows = shard_rows(4096, world, rank)
        enc_s = bitrl.Encoder(layers, 2560, 6912, 20, 5)
        hs = inputs.activations(4096, 2560, 6000)[row0:row0 + rows].contiguous().to(dev)
        hs_out = torch.empty_like(hs)
        ws_s = torch.empty((enc_s.workspace_bytes(rows),), dtype=torch.uint8, device=dev)
        gs_, _ = capture(lambda: enc_s.forward(hs, h_out=hs_out, workspace=ws_s))
        ms_s = time_graph(gs_, sub_steps, args.warmup, world) / sub_steps
        extra[f"encoder_{n_layers}_blocks_T4096_rows_sharded_x{world}"] = {
            "ms": ms_s, "states_per_s": 128.0 / (ms_s * 1e-3), "rows_per_rank": rows, "scaling": "strong"}
        del gs_, enc_s, hs, hs_out, ws_s

    if rank == 0 and "encoder" in sections:
        T = 4096  # 128 states x 32 tokens
        enc = bitrl.Encoder(layers, 2560, 6912, 20, 5)
        h0 = inputs.activations(T, 2560, 6000).to(dev)
        h1 = torch.empty_like(h0)
        ews = torch.empty((enc.workspace_bytes(T),), dtype=torch.uint8, device=dev)
        ge, le = capture(lambda: enc.forward(h0, h_out=h1, workspace=ews))
        mse = time_graph(ge, sub_steps, args.warmup, 1) / sub_steps
        enc_ops = 2.0 * T * sum(k * n for _, k, n in BLOCK) * n_layers
        i8_sus = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
        i8_burst = peaks["bf16_tflops"] * INT8_OVER_BF16
        enc_tops = enc_ops / (mse * 1e-3) / 1e12
        extra[f"encoder_{n_layers}_blocks_T4096"] = {
            "states_per_s": 128.0 / (mse * 1e-3), "ms": mse, "TOPS": enc_tops,
            "frac_of_int8_peak_sustained": enc_tops / i8_sus, "frac_of_int8_peak_burst": enc_tops / i8_burst,
            "frac_of_nominal_4500": enc_tops / 4500.0, "launches": le}
        del ge
        # the same stack with real attention inside each state: equal 32-token states, then ragged 15-40-token ones
        pooled = torch.empty((128, 2560), dtype=torch.bfloat16, device=dev)
        off = inputs.state_offsets(128, 7000)
        Tr = int(off[-1])
        cases = (("uniform32", T, 32, h0, h1),
                 ("ragged15to40", Tr, (off.to(torch.int32).to(dev), inputs.STATE_TOKENS_MAX),
                  inputs.activations(Tr, 2560, 6001).to(dev), torch.empty((Tr, 2560), dtype=torch.bfloat16, device=dev)))
        for label, Tc, states, hin, hout in cases:
            max_len = states if isinstance(states, int) else states[1]
            aws = torch.empty((enc.states_workspace_bytes(Tc, max_len),), dtype=torch.uint8, device=dev)
            ga, la = capture(lambda: enc.forward_states(hin, states, h_out=hout, pooled=pooled, workspace=aws))
            msa = time_graph(ga, sub_steps, args.warmup, 1) / sub_steps
            ops = 2.0 * Tc * sum(k * n for _, k, n in BLOCK) * n_layers
            extra[f"encoder_{n_layers}_blocks_attention_{label}"] = {
                "states_per_s": 128.0 / (msa * 1e-3), "ms": msa, "tokens": Tc, "bitlinear_TOPS": ops / (msa * 1e-3) / 1e12,
                "frac_of_int8_peak_sustained": ops / (msa * 1e-3) / 1e12 / i8_sus, "launches": la}
            del ga, aws
        # one agent step for 128 parallel environments: encoder with attention -> last-token latents -> policy and value
        # heads; then the update-side math on a 2048-step rollout of those environments (GAE) and a 64-sample mini-batch
        n_act = 6
        heads = [tuple(t.to(dev) for t in inputs.head_weights(2560, n_act, 8200)),
                 tuple(t.to(dev) for t in inputs.head_weights(2560, 1, 8201))]
        aws = torch.empty((enc.states_workspace_bytes(T, 32),), dtype=torch.uint8, device=dev)

        def agent_step():
            enc.forward_states(h0, 32, h_out=h1, pooled=pooled, workspace=aws)
            return bitrl.heads_forward(pooled, heads)

        gs, ls = capture(agent_step)
        mss = time_graph(gs, sub_steps, args.warmup, 1) / sub_steps
        extra["agent_step_128_states_x32_tokens"] = {"ms": mss, "states_per_s": 128.0 / (mss * 1e-3), "launches": ls}
        del gs
        # the paper's own operating point: ONE environment, one state of 32 tokens per step (latency, not throughput)
        h_one = inputs.activations(32, 2560, 6002).to(dev)
        h_one_out = torch.empty_like(h_one)
        pooled_one = torch.empty((1, 2560), dtype=torch.bfloat16, device=dev)
        ws_one = torch.empty((enc.states_workspace_bytes(32, 32),), dtype=torch.uint8, device=dev)

        def agent_step_one():
            enc.forward_states(h_one, 32, h_out=h_one_out, pooled=pooled_one, workspace=ws_one)
            return bitrl.heads_forward(pooled_one, heads)

        g1s, l1s = capture(agent_step_one)
        ms1s = time_graph(g1s, sub_steps, args.warmup, 1) / sub_steps
        extra["agent_step_1_state_x32_tokens"] = {"ms": ms1s, "launches": l1s,
                                                  "context": "the paper reports 24.8 ms median per step on a Raspberry Pi 4"}
        del g1s
        r, v, dn = (t.to(dev) for t in inputs.rollout(2048, 128, 8300))
        batch = [t.to(dev) for t in inputs.ppo_batch(64, n_act, 8400)]

        def update_math():
            bitrl.gae(r, v, dn)
            bitrl.ppo_loss(*batch)

        gu, lu = capture(update_math)
        msu = time_graph(gu, sub_steps, args.warmup, 1) / sub_steps
        extra["gae_2048x128_plus_ppo_loss_64"] = {"us": msu * 1e3, "launches": lu}
        del gu
    bitrl.poll_status()
    clocks_sections = sampler2.stop() if sampler2 else None
    cpu_other = None
    if rank == 0 and "cpu" in sections:
        cpu = oracle_decode_sample()
        cpu_other = oracle_batched_samples()

    if rank == 0:
        achieved = gbs1 / world
        line = {
            "metric": METRIC, "value": gbs1, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms1 / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8 x ternary(2-bit) -> int32", "data": "synthetic",
            "config": {"workload": f"configs[1]: decode GEMV sweep at M=1 over {n_layers} blocks x (2560->3840, "
                                   "2560->2560, 2560->13824, 6912->2560) of a ~2B BitNet b1.58 backbone; the "
                                   f"{4 * n_layers} independent GEMVs of a step go through the grouped entry point",
                       "launches_per_step": launches1, "packed_bytes_per_step": bytes_step,
                       "l2": f"{bytes_step / 1e6:.0f} MB of distinct weights per step against a 126 MB L2: inputs "
                             "larger than L2, no flush needed",
                       "timing": "one CUDA graph of the K steps (one grouped launch each, joined by programmatic dependent "
                                 "launch), launched once untimed after the W warm-up steps, then timed with CUDA events on the "
                                 "launching stream",
                       "parallelism": f"replicas x{world}, no collective"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"],
                         "traffic": None if HEADLINE_TRAFFIC_PER_BLOCK is None else HEADLINE_TRAFFIC_PER_BLOCK * n_layers, "peak_source": f"of {peak_src}",
                         "kernel": "gemv_multi_dp4a_kernel<1>", "us_per_launch": us_per_launch,
                         "algorithmic_bytes_per_launch": bytes_step / launches1,
                         "ms_per_step_spread": spread1,
                         "ms_per_step_one_graph_launch_per_step": ms1_single / args.steps,
                         "per_call_m1": per_call_m1, "gemm": gemm_roofline},
            "cpu_baseline": cpu,
            "cpu_baseline_batched": cpu_other,
            "e2e": {"value": e2e_gbs, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / args.steps,
                    "how": "each step = one graph (copy in, sweep, copy all outputs out) and a wait for its result",
                    "two_steps_in_flight": {"value": e2e_pipe_gbs, "ms_per_step": e2e_pipe_ms / args.steps,
                                            "how": "the same steps on two streams with two buffer sets: a step's "
                                                   "copies overlap the next step's kernel"}},
            "gpu_launches": launches_k,
            "clocks": clocks,
            "clocks_secondary_sections": clocks_sections,
            "extra": extra,
        }
        print(json.dumps(line))
    if world > 1:
        torch.distributed.barrier()  # the other ranks wait for rank 0's secondary sections before tearing down
        torch.distributed.destroy_process_group()


def free_port() -> int:
    import socket

    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def self_launch(n: int) -> int:
    """Re-runs this command line as n ranks (one process per GPU) on this node through torch.distributed.run; the
    ranks' output passes through, so rank 0's JSON line is this process's JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=FULL_LAYERS, help="blocks in the backbone (30 = full model)")
    ap.add_argument("--sections", default="decode8,pack,pack5,gemm,critic,encoder,cpu",
                    help="secondary measurements besides the M=1 headline (comma list; empty = none)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(self_launch(args.gpus))  # started as plain `python bench.py --gpus N`: become N ranks
    if args.impl == "reference":
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
