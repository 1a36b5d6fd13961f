#!/usr/bin/env python
"""Benchmark of the BNN run-time path on B200.

One step = one forward pass of the MNIST-shaped BNN MLP (Algorithm 4) over a batch of 10000 synthetic
images: bit-plane first layer, two fused binary 4096x4096 layers, real-valued 10-way output layer.
`value` is images/s with the batch resident in HBM; `e2e` is the same through bnn_mlp_forward_host
with pinned HOST buffers (copies inside the timed region).  The line also carries the binary-GEMM
throughput (8192^3, Tbit-op/s), the roofline of the dominant kernel, and the CPU oracle timed on the
host cores (`cpu_baseline`).  `--impl reference` times the oracle alone.

N > 1 (under torchrun): every rank runs its own batch (independent rows, no data-path collective);
time is the max over ranks and value the total images / that time.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

BATCH = 10000
SIZES = (784, 4096, 4096, 4096, 10)
SEED = 1
METRIC = "bnn_mlp_images_per_s"
UNIT = "images/s"
# Plain popc roofline: SMs x POPC lanes/clk/SM x 32 bit-MACs x 2 ops x max SM clock.  The POPC rate is measured in the
# same process (bnn_measure_pipe_rates); this documented figure is only the cross-check printed beside it.
POPC_PER_CLK_PER_SM_DOCUMENTED = 16
L2_FLUSH_BYTES = 256 << 20
SOAK_SECONDS = 0.6


def bit_ops_mlp(batch, sizes):
    """2 x bit-MACs of one forward pass, counting true K bits (8 planes for the first layer)."""
    ops = 2 * 8 * batch * sizes[0] * sizes[1]
    for k in range(1, len(sizes) - 1):
        ops += 2 * batch * sizes[k] * sizes[k + 1]
    return ops


class ClockSampler:
    """nvidia-smi sampling of SM clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [s for s, p in zip(sm, pw) if p >= 0.5 * max(pw)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "power_w_median": statistics.median([p for p in pw if p >= 0.5 * max(pw)] or pw),
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle_mlp(case, sample, repeats=1):
    import oracle
    oracle.build()
    X = case["X"][:sample]
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.mlp_forward(X, case["weights"], case["bns"])
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return best, oracle.host_threads()


def run_reference(args):
    """The CPU oracle as it stands, on the host cores: each step is the MLP forward on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_1602_02830_b200 import workloads as wl
    case = wl.mlp_case(batch=BATCH, sizes=SIZES, seed=SEED)
    sample = 1000
    for _ in range(max(args.warmup, 1)):
        time_oracle_mlp(case, min(sample, 200))
    times = []
    cores = 0
    for _ in range(args.steps):
        dt, cores = time_oracle_mlp(case, sample)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = sample / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32", "data": "synthetic",
            "config": {"workload": "MNIST-shaped BNN MLP 784-4096-4096-4096-10, seed 1; each step = %d of the 10000 images" % sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "%d images per step, %d steps" % (sample, args.steps)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def lib_dense_expanded(ctx, A_exp, W_exp, bits, thr, flip, out, M, N, K):
    """bnn_binary_dense_expanded into a preallocated packed output (no allocation inside the timed call)."""
    from paper_1602_02830_b200 import binding
    L = binding.lib()
    ptr = lambda t: None if t is None else ctypes.c_void_p(t.data_ptr())
    st = L.bnn_binary_dense_expanded(ctx._h, ptr(A_exp), A_exp.stride(0) * A_exp.element_size(), ptr(W_exp),
                                     W_exp.stride(0) * W_exp.element_size(), bits, ptr(thr), ptr(flip), ptr(out), out.stride(0),
                                     None, 0, M, N, K)
    if st != 0:
        raise RuntimeError("bnn_binary_dense_expanded failed: %d" % st)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--variant", type=int, default=0, help="tiled-kernel inner loop: 0 default, 1 plain popc, 2 carry-save")
    ap.add_argument("--engine", type=int, default=0, help="0 auto (tensor-core engine for large shapes), 1 CUDA-core XOR-popcount only, 2 tensor")
    ap.add_argument("--tile-rows", type=int, default=0, help="accumulator rows per thread of the CUDA-core tile kernel (8 or 16; 0 = library default)")
    ap.add_argument("--pair-mode", type=int, default=0, help="tensor engine CTA pairs (cta_group::2): 0 = for very large outputs, 1 = never, 2 = wherever possible")
    ap.add_argument("--operand-bits", type=int, default=4, choices=[4, 8],
                    help="tensor engine, +-1 x +-1 products: 4 = e2m1 nibbles (kind::mxf4), 8 = signed bytes (kind::i8)")
    ap.add_argument("--conv-form", type=int, default=0, choices=[0, 1], help="tensor engine convolutions: 0 halo tiles, 1 one operand box per tap")
    ap.add_argument("--no-extras", action="store_true", help="skip the side measurements (configs, ConvNet, Fig. 3) and the CPU baseline")
    ap.add_argument("--gemm-size", type=int, default=8192)
    ap.add_argument("--section", default="all", choices=["all", "gemm", "convnet", "sweep", "fig3", "configs"],
                    help="side measurements to run after the MLP step (a single one keeps profiler captures small)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_1602_02830_b200 import binding, build, nets, replicas, workloads as wl

    world, rank, local = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    replicas.init("nccl", torch.device("cuda", local))
    if rank == 0:
        build.build()
    replicas.barrier()
    dev = f"cuda:{local}"
    stream = torch.cuda.current_stream(local)
    ctx = binding.Context(local, stream)
    ctx.set_popc_variant(args.variant)
    ctx.set_engine(args.engine)
    if args.tile_rows:
        ctx.set_tile_rows(args.tile_rows)
    ctx.set_pair_mode(args.pair_mode)
    ctx.set_operand_bits(args.operand_bits)
    ctx.set_conv_form(args.conv_form)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            replicas.barrier()
            torch.cuda.synchronize()

    # ---- workload: every rank draws the same network; rank r gets its own batch of images
    case = wl.mlp_case(batch=BATCH, sizes=SIZES, seed=SEED)
    if rank > 0:
        case["X"] = wl.u8(np.random.default_rng(replicas.rank_seed(SEED, rank)), (BATCH, SIZES[0]))
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    desc = net["desc"]
    ws = torch.empty(ctx.mlp_workspace_bytes(desc, BATCH, True), dtype=torch.uint8, device=dev)
    ctx.set_workspace(ws)
    X = torch.from_numpy(case["X"]).to(dev)
    scores = torch.empty(BATCH, SIZES[-1], dtype=torch.float32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tensor_step = args.engine != 1          # batch 10000 qualifies for the tensor engine on every hidden layer
    # per step: one kernel per layer on either engine
    # (weights are expanded to bytes once, outside the step, like packing and the BatchNorm fold)
    launches_per_step = len(SIZES) - 1

    def timed_steps(fn, steps, warmup):
        """CUDA events on the launch stream around each step; L2 flushed (untimed) before each step."""
        for _ in range(warmup):
            flush.fill_(1)
            fn()
        sync_all()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.fill_(1)
            a.record(stream)
            fn()
            b.record(stream)
        sync_all()
        return [a.elapsed_time(b) for a, b in ev]

    def median_ms(fn, steps=20, warmup=3):
        t = timed_steps(fn, steps, warmup)
        return sorted(t)[len(t) // 2]

    step_fn = lambda: ctx.mlp_forward(desc, X, BATCH, scores=scores)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.15)                     # nvidia-smi needs ~0.1 s before its first sample
    times = timed_steps(step_fn, args.steps, args.warmup)
    total_ms = sum(times)
    # the clock record belongs to the timed region above; the poller is stopped before the end-to-end loop because its
    # driver queries slow down host<->device copies issued meanwhile
    clocks = sampler.stop() if sampler else None

    # ---- soak: the same step back to back (no flush, no gaps) for at least SOAK_SECONDS, with its own clock record:
    # the sustained figure under load, next to the counted steps above whose timed region lasts only milliseconds
    soak = None
    if rank == 0:
        n_soak = max(200, int(SOAK_SECONDS * 1e3 / max(total_ms / args.steps, 1e-3)))
        sampler2 = ClockSampler(local)
        sampler2.start()
        time.sleep(0.05)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_soak):
            step_fn()
        e1.record(stream)
        torch.cuda.synchronize()
        soak_ms = e0.elapsed_time(e1) / n_soak
        soak = {"steps": n_soak, "seconds": e0.elapsed_time(e1) / 1e3, "ms_per_step": soak_ms,
                "images_per_s": BATCH / (soak_ms / 1e3), "clocks": sampler2.stop(),
                "note": "back to back, working set stays in L2 (no flush between steps)"}

    if clocks is not None and clocks.get("sm_mhz") is None and soak is not None and soak["clocks"].get("sm_mhz") is not None:
        # the counted region (a few milliseconds) fell between two samples: the record of the soak (the same step, back to
        # back, right after it) stands in and says so
        clocks = dict(soak["clocks"], source="soak: the counted region was shorter than one sampling period")

    # ---- end to end: pinned host buffers, copies inside the timed region
    Xh = torch.from_numpy(case["X"]).pin_memory()
    Sh = torch.empty(BATCH, SIZES[-1], dtype=torch.float32).pin_memory()
    # Warm-up until steady, whatever --steps says: on these hosts the copy path (PCIe link / host uncore clocks) needs
    # several hundred ms of traffic before the transfer time settles (0.86 -> 0.43 ms per step over the first ~400 steps),
    # so blocks of 100 steps run until a block is within 2 % of the one before it AND of the fastest block so far (at most
    # 30 blocks, ~1 s).
    e2e_fn = lambda: ctx.mlp_forward_host(desc, Xh, BATCH, Sh)
    prev, best, e2e_warm_blocks = None, None, 0
    for _ in range(30):
        blk = sum(timed_steps(e2e_fn, 100, 0)) / 100
        e2e_warm_blocks += 1
        steady = prev is not None and abs(blk - prev) <= 0.02 * prev and blk <= 1.02 * best
        best = blk if best is None else min(best, blk)
        prev = blk
        if steady and e2e_warm_blocks >= 5:
            break
    e2e_times = timed_steps(e2e_fn, max(args.steps, 50), max(args.warmup, 3))
    e2e_total_ms = sum(e2e_times) * args.steps / len(e2e_times)       # scaled to --steps steps
    if os.environ.get("BNN_BENCH_DEBUG"):
        print("e2e per-step ms:", " ".join("%.3f" % t for t in e2e_times), file=sys.stderr)

    # ---- dominant kernel of the step, timed alone on the same stream: the fused 4096x4096 binary dense layer
    hid = net["layers"][1]
    dcase = wl.dense_case(BATCH, K=SIZES[1], N=SIZES[2], seed=4)      # seeded +-1 activations of the layer's shape
    act_in = ctx.pack_signs(torch.from_numpy(dcase["A"]).to(dev))
    act_out = torch.empty(BATCH, binding.packed_ld(SIZES[2]), dtype=torch.int32, device=dev)
    dense_times = timed_steps(lambda: ctx.binary_dense(act_in, hid["Wp"], hid["thr"], hid["flip"], BATCH, SIZES[2], SIZES[1],
                                                       out=act_out), min(args.steps, 50), 3)
    # ... and the tensor kernel of that layer by itself, on operands that are already expanded (what runs inside the step,
    # where the weights were expanded once and the previous layer wrote the activations in operand format)
    kernel_ms, kernel_name, kernel_clock = None, None, (None, None)
    if tensor_step:
        bits = args.operand_bits
        expand = ctx.expand_signs_f4 if bits == 4 else ctx.expand_signs
        A_exp = expand(act_in, BATCH, SIZES[1])
        W_exp = expand(hid["Wp"], SIZES[2], SIZES[1])
        kernel_times = timed_steps(lambda: lib_dense_expanded(ctx, A_exp, W_exp, bits, hid["thr"], hid["flip"], act_out, BATCH,
                                                              SIZES[2], SIZES[1]), min(args.steps, 50), 3)
        kernel_ms = sum(kernel_times) / len(kernel_times)
        kernel_name = ctx.last_tensor_kernel()
        kernel_clock = ctx.last_tensor_kernel_clock()      # (SM MHz inside the last launch, us its first CTA lived)
        del A_exp, W_exp
    first = net["layers"][0]
    first_times = timed_steps(lambda: ctx.first_layer_bitplanes(X, first["Wp"], BATCH, SIZES[1], SIZES[0], thr=first["thr"],
                                                                flip=first["flip"]), min(args.steps, 50), 3)
    first_kernel_name = ctx.last_tensor_kernel() if tensor_step else "k_bit_tile (bit-plane operand)"

    total_ms, e2e_total_ms = replicas.max_over_ranks([total_ms, e2e_total_ms], device=dev)
    ms_per_step = total_ms / args.steps
    value = replicas.job_throughput(BATCH, ms_per_step, world)
    e2e_value = replicas.job_throughput(BATCH, e2e_total_ms / args.steps, world)

    if rank != 0:
        replicas.finish()
        return 0

    # ---- the roofline denominators of this run
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    rates = ctx.measure_pipe_rates()                  # POPC / LOP3 / xor+popc+add results per clock and SM, measured now
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    sm_max_mhz = float(peaks.get("sm_max_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0)
    popc_peak_tbitops = sm_count * rates["popc"] * 32 * 2 * sm_max_mhz * 1e6 / 1e12
    bf16_peak = float(peaks.get("bf16_tflops") or 1590.0)
    bf16_sustained = float(peaks.get("bf16_tflops_sustained") or 1400.0)
    # nominal dense ratios to bf16 (2.25 PFLOP/s): int8 4.5 -> 2x, fp4 9 -> 4x
    peak_ratio = 4.0 if args.operand_bits == 4 else 2.0
    tensor_peak = peak_ratio * bf16_peak
    which = "of measured" if peaks else "of fallback"

    # the same two layers on the CUDA-core XOR-popcount path (Eq. 8 as the paper computes it), for the popc roofline
    ctx.set_engine(1)
    popc_dense_times = timed_steps(lambda: ctx.binary_dense(act_in, hid["Wp"], hid["thr"], hid["flip"], BATCH, SIZES[2], SIZES[1],
                                                            out=act_out), min(args.steps, 20), 3)
    popc_mlp_times = timed_steps(step_fn, min(args.steps, 20), 3)
    ctx.set_engine(args.engine)

    dense_ms = sum(dense_times) / len(dense_times)
    dense_ops = 2.0 * BATCH * SIZES[1] * SIZES[2]
    dense_ach = dense_ops / (dense_ms / 1e3) / 1e12
    popc_dense_ms = sum(popc_dense_times) / len(popc_dense_times)
    popc_dense_ach = dense_ops / (popc_dense_ms / 1e3) / 1e12
    popc_mlp_ms = sum(popc_mlp_times) / len(popc_mlp_times)
    popc_mlp_ach = bit_ops_mlp(BATCH, SIZES) / (popc_mlp_ms / 1e3) / 1e12
    first_ms = sum(first_times) / len(first_times)
    # composite tensor roofline of the step: every layer's operations at the peak of the operand type it runs on
    # (first layer: bytes; hidden layers: nibbles or bytes; the 10-way output layer is 0.1 % of the work and left out)
    first_ops = 2.0 * BATCH * SIZES[0] * SIZES[1]
    hidden_ops = sum(2.0 * BATCH * SIZES[k] * SIZES[k + 1] for k in range(1, len(SIZES) - 2))
    ideal_step_ms = (first_ops / (2.0 * bf16_peak * 1e12) + hidden_ops / (tensor_peak * 1e12)) * 1e3
    ideal_soak_ms = (first_ops / (2.0 * bf16_sustained * 1e12) + hidden_ops / (peak_ratio * bf16_sustained * 1e12)) * 1e3
    if soak:
        soak["tensor_composite_frac_of_sustained"] = ideal_soak_ms / soak["ms_per_step"] if tensor_step else None
        soak["peak_kind"] = "per-layer ideal at the operand type's nominal multiple of the measured SUSTAINED bf16 rate %.1f TFLOP/s" % bf16_sustained

    first_what = ("u8 x s8 byte product on the tensor cores (the 8 bit-plane terms of Eq. 7 summed by the multiplier)" if tensor_step
                  else "8 bit-planes, AND-popcount")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": "MNIST-shaped BNN MLP forward 784-4096-4096-4096-10 (first layer: %s; 2 fused binary dense; float "
                               "output), batch 10000 per GPU, seed 1" % first_what,
                   "batch_per_gpu": BATCH, "parallelism": "replicas x%d" % world,
                   "l2": "256 MiB written between timed steps (inputs fit in L2)", "popc_variant": args.variant,
                   "operand_bits": args.operand_bits,
                   "engine": {0: "auto (tensor-core engine for the large layers)", 1: "CUDA-core XOR-popcount", 2: "tensor"}[args.engine]},
        "clocks": clocks,
        "soak": soak,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": BATCH * SIZES[0], "d2h_bytes_per_step": BATCH * SIZES[-1] * 4,
                "ms_per_step": e2e_total_ms / args.steps, "ms_median": statistics.median(e2e_times), "ms_min": min(e2e_times),
                "ms_max": max(e2e_times), "timed_steps": len(e2e_times), "warmup_steps": 100 * e2e_warm_blocks + max(args.warmup, 3)},
        "gpu_launches": launches_per_step * args.steps,
        "pipe_rates_measured": {"popc_per_clk_per_sm": rates["popc"], "lop3_per_clk_per_sm": rates["lop3"],
                                "xor_popc_add_words_per_clk_per_sm": rates["xor_popc_add"],
                                "popc_per_clk_per_sm_documented": POPC_PER_CLK_PER_SM_DOCUMENTED,
                                "clock_used_mhz": sm_max_mhz, "sm_count": sm_count, "popc_peak_tbitops": popc_peak_tbitops,
                                "how": "bnn_measure_pipe_rates in this process: register-only loops on every SM, clock64"},
        "roofline": ({"bound": "tensor", "kernel": "%s: the hidden layer 10000x4096x4096 of the step (bnn_binary_dense_expanded on "
                                                    "operands already in the tensor engine's format, as inside the step)" % kernel_name,
                      "achieved": dense_ops / (kernel_ms / 1e3) / 1e12, "peak": tensor_peak, "unit": "TFLOP/s",
                      "frac": dense_ops / (kernel_ms / 1e3) / 1e12 / tensor_peak,
                      "traffic": 28969984 if args.operand_bits == 4 else 60967424,
                      "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum of this kernel, one launch: "
                                        "profiles/k_umma_i8_mlp_batch10000.md (not re-measured by this run)",
                      "peak_kind": "2 ops per MAC; peak = %.0f x measured bf16 burst %.1f TFLOP/s (NOMINAL %s:bf16 ratio, not a "
                                   "measured %s rate), %s" % (peak_ratio, bf16_peak, "fp4" if args.operand_bits == 4 else "int8",
                                                              "mxf4" if args.operand_bits == 4 else "int8", which),
                      "frac_of_probe_rate": (dense_ops / (kernel_ms / 1e3) / 1e12 / 8857.0) if args.operand_bits == 4 else None,
                      "probe_rate_note": "8857 TOPS = kind::mxf4 with resident operands, all SMs, measured once on this pool "
                                         "(profiles/pipe_rates_sm100.md)",
                      "ms_per_launch": kernel_ms,
                      "sm_mhz_in_kernel": kernel_clock[0], "us_in_kernel_cta0": kernel_clock[1],
                      "sm_mhz_note": "clock64 against %globaltimer inside the last timed launch (bnn_last_tensor_kernel_clock): the "
                                     "clock the kernel ran at, as opposed to the maximum that nvidia-smi samples around it",
                      "fused_call": {"what": "bnn_binary_dense from packed operands: two expansion kernels + the same kernel",
                                     "ms": dense_ms, "achieved": dense_ach, "frac": dense_ach / tensor_peak}}
                     if tensor_step else
                     {"bound": "alu", "kernel": "k_bit_tile (fused binary dense 10000x4096x4096)", "achieved": dense_ach,
                      "peak": popc_peak_tbitops, "unit": "Tbit-op/s", "frac": dense_ach / popc_peak_tbitops, "traffic": 7299840,
                      "traffic_source": "ncu, profiles/k_bit_tile_mlp_batch10000.md (not re-measured by this run)",
                      "peak_kind": "derived: %d SMs x %.2f POPC/clk/SM (measured in this run) x 32 bit-MAC x 2 x %.0f MHz (one POPC "
                                   "per 32-bit word); carry-save kernels may exceed it" % (sm_count, rates["popc"], sm_max_mhz),
                      "ms_per_launch": dense_ms}),
        "popc_path": {"what": "the same layer and the same MLP step on the CUDA-core XOR-popcount kernels (engine 1): the path the "
                              "popcount roofline applies to",
                      "dense_layer_ms": popc_dense_ms, "dense_tbitops": popc_dense_ach,
                      "dense_frac_of_popc_peak": popc_dense_ach / popc_peak_tbitops,
                      "dense_frac_of_carry_save_ceiling": popc_dense_ach / (2 * popc_peak_tbitops),
                      "popc_peak_tbitops": popc_peak_tbitops,
                      "mlp_ms_per_step": popc_mlp_ms, "mlp_images_per_s": BATCH / (popc_mlp_ms / 1e3), "mlp_tbitops": popc_mlp_ach,
                      "mlp_frac": popc_mlp_ach / popc_peak_tbitops, "mlp_frac_of_carry_save_ceiling": popc_mlp_ach / (2 * popc_peak_tbitops),
                      "note": "bit-ops count 8 planes for the first layer; one POPC per word is the plain roofline, the carry-save "
                              "inner loop (one POPC per two words) has twice that ceiling"},
        "mlp_step": {"first_layer_ms": first_ms, "first_layer_kernel": first_kernel_name,
                     "first_layer_frac_of_int8_peak": (first_ops / (first_ms / 1e3) / 1e12) / (2.0 * bf16_peak) if tensor_step else None,
                     "dense_layer_ms": dense_ms, "dense_kernel_ms": kernel_ms,
                     "tensor_composite_ideal_ms": ideal_step_ms if tensor_step else None,
                     "tensor_composite_frac": (ideal_step_ms / ms_per_step) if tensor_step else None,
                     "x_popc_roofline_equivalent": bit_ops_mlp(BATCH, SIZES) / (ms_per_step / 1e3) / 1e12 / popc_peak_tbitops,
                     "note": "tensor_composite_frac = sum over layers of (2 MACs / nominal peak of the layer's operand type) / ms_per_step; "
                             "x_popc_roofline_equivalent is NOT a roofline fraction on the tensor engine: it says how many popcount "
                             "rooflines' worth of bit-ops per second the step delivers"},
    }

    if not args.no_extras and world == 1:
        sec = args.section
        if sec in ("all", "gemm", "configs"):
            line["configs"] = bench_configs(ctx, timed_steps, median_ms, args, popc_peak_tbitops, tensor_peak, peaks,
                                            full=(sec != "gemm"))
        if sec in ("all", "convnet"):
            line["convnet"] = bench_convnet(ctx, timed_steps, median_ms, args, bf16_peak)
        if sec in ("all", "sweep"):
            line["dense_sweep"] = bench_dense_sweep(ctx, timed_steps, median_ms, args.engine, args.operand_bits)
        if sec == "all":
            line["other_readings"] = bench_other_readings(ctx, median_ms)
            line["filter_repetition"] = bench_filter_repetition(ctx, median_ms, args.engine)
        if sec in ("all", "fig3"):
            line["fig3_context"] = bench_fig3(ctx, timed_steps, args.engine, popc_mlp_ms, ms_per_step)
        ctx.set_workspace(ws)
        t0 = time.perf_counter()
        dt, cores = time_oracle_mlp(case, BATCH, repeats=4 if sec == "all" else 1)
        line["cpu_baseline"] = {"value": BATCH / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": "the whole batch of 10000 images, best of %d passes (%.1f s of CPU work in total)"
                                          % (4 if sec == "all" else 1, time.perf_counter() - t0)}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    replicas.finish()
    return 0


def bench_fig3(ctx, timed_steps, engine, popc_mlp_ms, mlp_ms):
    """The paper's Fig. 3 on this GPU (context, not a target): 8192^3 product of +-1 matrices with (a) a deliberately
    unoptimized float32 kernel, (b) the XNOR-popcount kernel, (c) cuBLAS via torch.matmul; and the MLP with the
    unoptimized kernel in place of the binary one.  The paper reports XNOR 23x faster than its baseline kernel and
    3.4x faster than cuBLAS, and the MLP 7x faster, on a GTX750."""
    import torch
    from paper_1602_02830_b200 import workloads as wl
    n = 8192
    Ah, Bh = wl.gemm_case(n, n, n, seed=2)
    A, B = torch.from_numpy(Ah).cuda(), torch.from_numpy(Bh).cuda()
    Af, Bf = A.float(), B.float()
    C = torch.empty(n, n, dtype=torch.float32, device="cuda")
    base = timed_steps(lambda: ctx.baseline_gemm_f32(Af, Bf, C), 2, 1)
    base_ms = min(base)
    torch.backends.cuda.matmul.allow_tf32 = False
    cublas_f32 = min(timed_steps(lambda: torch.matmul(Af, Bf, out=C), 3, 2))
    Ab, Bb = A.to(torch.bfloat16), B.to(torch.bfloat16)
    Cb = torch.empty(n, n, dtype=torch.bfloat16, device="cuda")
    cublas_bf16 = min(timed_steps(lambda: torch.matmul(Ab, Bb, out=Cb), 5, 3))
    try:
        cublas_i8 = min(timed_steps(lambda: torch._int_mm(A, B), 5, 3))
    except Exception:  # pragma: no cover - library support varies
        cublas_i8 = None
    Ap = ctx.pack_signs(A)
    Bp = ctx.pack_signs(B, pack_along=1)
    Ci = torch.empty(n, n, dtype=torch.int32, device="cuda")
    ctx.set_engine(1)
    xnor_ms = min(timed_steps(lambda: ctx.xnor_gemm(Ap, Bp, n, n, n, C=Ci), 5, 3))
    ctx.set_engine(engine)
    assert torch.equal(Ci.float(), torch.matmul(Af, Bf)), "XNOR kernel and float product differ"   # fp32 is exact here
    del Ab, Bb, Cb, Ci
    # MLP with the unoptimized float kernel standing in for every layer's product (batch 10000, same shapes)
    mlp_base = 0.0
    for K, N in zip(SIZES[:-1], SIZES[1:]):
        X = torch.ones(BATCH, K, dtype=torch.float32, device="cuda")
        W = torch.ones(K, N, dtype=torch.float32, device="cuda")
        O = torch.empty(BATCH, N, dtype=torch.float32, device="cuda")
        mlp_base += min(timed_steps(lambda: ctx.baseline_gemm_f32(X, W, O), 2, 1))
    return {"shape": [n, n, n], "baseline_f32_ms": base_ms, "xnor_popc_ms": xnor_ms, "cublas_f32_ms": cublas_f32,
            "cublas_bf16_ms": cublas_bf16, "cublas_int8_ms": cublas_i8,
            "xnor_vs_baseline": base_ms / xnor_ms, "xnor_vs_cublas_f32": cublas_f32 / xnor_ms,
            "mlp_baseline_kernel_ms": mlp_base, "mlp_xnor_vs_baseline": mlp_base / popc_mlp_ms,
            "mlp_selected_engine_vs_baseline": mlp_base / mlp_ms,
            "paper_gtx750": {"xnor_vs_baseline": 23, "xnor_vs_cublas": 3.4, "mlp_xnor_vs_baseline": 7}}


def launch_floor_ms(ctx, median_ms):
    """A one-word sign-pack (one tiny kernel) timed like everything else: what any single call costs at least."""
    import torch
    tiny_src = torch.zeros(1, 32, dtype=torch.int8, device="cuda")
    tiny_dst = torch.empty(1, 4, dtype=torch.int32, device="cuda")
    return median_ms(lambda: ctx.pack_signs(tiny_src, dst=tiny_dst))


def bench_dense_sweep(ctx, timed_steps, median_ms, engine, operand_bits):
    """Configuration 5: one fused 4096 -> 4096 binary dense layer at batch 1 .. 65536 (seed 4, thresholds uniform in
    [-64, 64]) on the CUDA-core kernels, on the selected engine from packed operands (expansion passes inside the time) and,
    where the tensor engine applies, on operands kept in its format (bnn_binary_dense_expanded)."""
    import torch
    from paper_1602_02830_b200 import binding, workloads as wl
    K = N = 4096
    out = {"launch_floor_ms": launch_floor_ms(ctx, median_ms)}
    base = wl.dense_case(1)
    Wp = ctx.pack_signs(torch.from_numpy(base["W"]).cuda(), pack_along=1)
    thr = torch.from_numpy(base["thr"]).cuda()
    expand = ctx.expand_signs_f4 if operand_bits == 4 else ctx.expand_signs
    W_exp = expand(Wp, N, K)
    for batch in wl.DENSE_BATCHES:
        Ap = ctx.pack_signs(torch.from_numpy(wl.dense_case(batch)["A"]).cuda())
        O = torch.empty(batch, N // 32, dtype=torch.int32, device="cuda")
        dws = torch.empty(max(ctx.gemm_workspace_bytes(batch, N, K), 256), dtype=torch.uint8, device="cuda")
        ctx.set_workspace(dws)
        row = {}
        for name, eng in (("popc", 1), ("selected_engine", engine)):
            ctx.set_engine(eng)
            ms = median_ms(lambda: ctx.binary_dense(Ap, Wp, thr, None, batch, N, K, out=O))
            row[name] = {"ms": ms, "tbitops": 2.0 * batch * N * K / (ms / 1e3) / 1e12}
        ctx.set_engine(engine)
        if engine != 1 and ctx.gemm_workspace_bytes(batch, N, K) > 0:
            A_exp = expand(Ap, batch, K)
            ms = median_ms(lambda: lib_dense_expanded(ctx, A_exp, W_exp, operand_bits, thr, None, O, batch, N, K))
            row["expanded_operands"] = {"ms": ms, "tbitops": 2.0 * batch * N * K / (ms / 1e3) / 1e12}
            del A_exp
        out[str(batch)] = row
        ctx.set_workspace(None)
        del dws, Ap, O
    return out


def bench_configs(ctx, timed_steps, median_ms, args, popc_peak, tensor_peak, peaks, full=True):
    """The configurations the metric names, with their seeded inputs (workloads.py): the single small GEMM, the square sweep
    plus the ragged case on both engines (from packed operands to int32 sums), and bnn_pack_signs against the HBM rate."""
    import torch
    from paper_1602_02830_b200 import workloads as wl
    out = {"launch_floor_ms": launch_floor_ms(ctx, median_ms)}
    engine = args.engine
    # configuration 1: 64 x 512 times 512 x 256
    A, B = wl.config1()
    Ap = ctx.pack_signs(torch.from_numpy(A).cuda())
    Bp = ctx.pack_signs(torch.from_numpy(B).cuda(), pack_along=1)
    C = torch.empty(64, 256, dtype=torch.int32, device="cuda")
    out["cfg1_gemm_64x512x256"] = {"ms": median_ms(lambda: ctx.xnor_gemm(Ap, Bp, 64, 256, 512, C=C), 50, 5),
                                   "note": "launch / latency bound: compare with launch_floor_ms"}
    # configuration 3 (or just --gemm-size for a profiler capture)
    shapes = wl.GEMM_SWEEP if full else [(args.gemm_size,) * 3]
    sweep = {}
    for (M, N, K) in shapes:
        A, B = wl.gemm_case(M, N, K, seed=2)
        Ap = ctx.pack_signs(torch.from_numpy(A).cuda())
        Bp = ctx.pack_signs(torch.from_numpy(B).cuda(), pack_along=1)
        del A, B
        C = torch.empty(M, N, dtype=torch.int32, device="cuda")
        gws = torch.empty(max(ctx.gemm_workspace_bytes(M, N, K), 256), dtype=torch.uint8, device="cuda")
        ctx.set_workspace(gws)
        row = {}
        for name, eng in (("popc", 1), ("selected_engine", engine)):
            ctx.set_engine(eng)
            t = timed_steps(lambda: ctx.xnor_gemm(Ap, Bp, M, N, K, C=C), 5, 3)
            ms = sum(t) / len(t)
            tb = 2.0 * M * N * K / (ms / 1e3) / 1e12
            row[name] = {"ms": ms, "tbitops": tb}
            if eng == 1:
                row[name]["frac_of_popc_peak"] = tb / popc_peak
                row[name]["frac_of_carry_save_ceiling"] = tb / (2 * popc_peak)
            else:
                row[name]["frac_of_tensor_peak"] = tb / tensor_peak          # expansion passes inside the time
                row[name]["kernel"] = ctx.last_tensor_kernel()
                row[name]["x_popc_roofline_equivalent"] = tb / popc_peak
        sweep["%dx%dx%d" % (M, N, K)] = row
        ctx.set_workspace(None)
        del gws, C, Ap, Bp
    ctx.set_engine(engine)
    out["cfg3_gemm_sweep"] = sweep
    if full:
        # bnn_pack_signs, 16384 x 16384 elements, against the measured HBM copy rate (bytes read + bytes written)
        hbm = float(peaks.get("hbm_gbs") or 6650.0)
        n = 16384
        src8 = torch.from_numpy(wl.gemm_case(n, 1, n, seed=2)[0]).cuda()
        dst = torch.empty(n, n // 32, dtype=torch.int32, device="cuda")
        pack = {}
        for name, src in (("int8", src8), ("float16", src8.half()), ("float32", src8.float())):
            ms = median_ms(lambda: ctx.pack_signs(src, dst=dst), 10, 3)
            gbs = (src.numel() * src.element_size() + dst.numel() * 4) / (ms / 1e3) / 1e9
            pack[name] = {"ms": ms, "gb_per_s": gbs, "frac_of_hbm_copy": gbs / hbm}
            del src
        pack["hbm_gbs"] = hbm
        pack["peak_kind"] = "measured copy bandwidth, %s" % ("of measured" if peaks else "of fallback")
        out["pack_signs_16384x16384"] = pack
    return out


def conv_layer_ideal_ms(batch, hw, layers, bf16_peak, operand_bits):
    """Dense-count MACs of every layer at the nominal peak of the operand type it runs on (bytes for the 8-bit first layer and for
    layers whose C_in is not a multiple of 256, nibbles otherwise)."""
    out = []
    h = hw
    for i, L in enumerate(layers):
        cout, _, _, cin = L["wgt"].shape
        macs = batch * h * h * 9 * cin * cout
        ratio = 4.0 if (i > 0 and operand_bits == 4 and cin % 256 == 0) else 2.0
        out.append(2.0 * macs / (ratio * bf16_peak * 1e12) * 1e3)
        if L["pool"]:
            h //= 2
    return out


def bench_convnet(ctx, timed_steps, median_ms, args, bf16_peak):
    """Configuration 4: CIFAR-shaped ConvNet forward, batch 256, through bnn_convnet_forward: images/s on both engines, the
    composite tensor roofline of the selected engine, and per-layer times as differences of the forward pass over the first
    k layers (k = 1 .. 6)."""
    import torch
    from paper_1602_02830_b200 import nets, workloads as wl
    engine = args.engine
    case = wl.convnet_case()
    B, hw = case["batch"], case["hw"]
    net = nets.prepare_convnet(ctx, case["layers"])
    X = torch.from_numpy(case["X"]).cuda()
    desc, keep = ctx.make_convnet_desc(net)
    cws = torch.empty(max(ctx.convnet_workspace_bytes(desc, B, hw, hw), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(cws)
    final = torch.empty(nets.convnet_output_shape(net, B, hw, hw), dtype=torch.int32, device="cuda")
    out = {"batch": B}
    for name, eng in (("popc", 1), ("selected_engine", engine)):
        ctx.set_engine(eng)
        t = timed_steps(lambda: ctx.convnet_forward(desc, X, B, hw, hw, final), 20, 3)
        ms = sum(t) / len(t)
        out[name] = {"ms": ms, "images_per_s": B / (ms / 1e3)}
    ctx.set_engine(engine)
    if engine != 1:
        ideal = conv_layer_ideal_ms(B, hw, case["layers"], bf16_peak, args.operand_bits)
        prefix_ms, kernels = [], []
        for k in range(1, len(net) + 1):
            dk, keep_k = ctx.make_convnet_desc(net[:k])
            fk = torch.empty(nets.convnet_output_shape(net[:k], B, hw, hw), dtype=torch.int32, device="cuda")
            prefix_ms.append(median_ms(lambda: ctx.convnet_forward(dk, X, B, hw, hw, fk)))
            kernels.append(ctx.last_tensor_kernel())
        per_layer = [prefix_ms[0]] + [prefix_ms[k] - prefix_ms[k - 1] for k in range(1, len(prefix_ms))]
        ms = out["selected_engine"]["ms"]
        out["selected_engine"].update({
            "ideal_ms": sum(ideal), "frac": sum(ideal) / ms, "layer_ideal_ms": ideal, "layer_ms": per_layer,
            "layer_frac": [i / t if t > 0 else None for i, t in zip(ideal, per_layer)], "layer_kernel": kernels,
            "conv_form": "halo tiles" if args.conv_form == 0 else "one operand box per tap",
            "peak_kind": "dense-count MACs x 2 / (2 x bf16 burst for byte layers, 4 x for nibble layers): nominal ratios of the "
                         "measured bf16 burst %.1f TFLOP/s" % bf16_peak,
            "layer_ms_how": "median forward time over the first k layers minus that over the first k - 1 (the first layer's figure "
                            "includes its im2col pass)"})
    ctx.set_workspace(None)
    return out


def bench_other_readings(ctx, median_ms):
    """The other literal readings of the two network configurations and the ConvNet with its fully-connected tail: same calls,
    other layer lists (secondary rows; the headline keeps the paper's topology)."""
    import torch
    from paper_1602_02830_b200 import binding, nets, workloads as wl
    out = {}
    # MLP with one more 4096 x 4096 layer
    sizes = (784, 4096, 4096, 4096, 4096, 10)
    case = wl.mlp_case(batch=BATCH, sizes=sizes, seed=21)
    net = nets.prepare_mlp(ctx, case["weights"], case["bns"])
    ws = torch.empty(ctx.mlp_workspace_bytes(net["desc"], BATCH, False), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    X = torch.from_numpy(case["X"]).cuda()
    S = torch.empty(BATCH, 10, dtype=torch.float32, device="cuda")
    ms = median_ms(lambda: ctx.mlp_forward(net["desc"], X, BATCH, scores=S))
    out["mlp_784_4x4096_10_batch10000"] = {"ms": ms, "images_per_s": BATCH / (ms / 1e3)}
    ctx.set_workspace(None)
    del ws, net, X
    # ConvNet with one more 128 -> 128 convolution (seven convolutions, pools after the 3rd, 5th and 7th)
    B, hw = 256, 32
    case = wl.convnet_case(batch=B, channels=(128, 128, 128, 256, 256, 512, 512), seed=22)
    for i, L in enumerate(case["layers"]):
        L["pool"] = i in (2, 4, 6)
    cnet = nets.prepare_convnet(ctx, case["layers"])
    desc, keep = ctx.make_convnet_desc(cnet)
    cws = torch.empty(max(ctx.convnet_workspace_bytes(desc, B, hw, hw), 256), dtype=torch.uint8, device="cuda")
    ctx.set_workspace(cws)
    Xc = torch.from_numpy(case["X"]).cuda()
    final = torch.empty(nets.convnet_output_shape(cnet, B, hw, hw), dtype=torch.int32, device="cuda")
    ms = median_ms(lambda: ctx.convnet_forward(desc, Xc, B, hw, hw, final))
    out["convnet_7_convolutions_batch256"] = {"ms": ms, "images_per_s": B / (ms / 1e3)}
    # the paper's six-convolution net followed by 8192 -> 1024 -> 1024 -> 10 on the flattened map
    case = wl.convnet_case(batch=B, seed=23)
    cnet = nets.prepare_convnet(ctx, case["layers"])
    desc, keep = ctx.make_convnet_desc(cnet)
    rng = np.random.default_rng(24)
    K = 4 * 4 * 512
    W1, W2, W3 = wl.pm1(rng, (K, 1024)), wl.pm1(rng, (1024, 1024)), wl.pm1(rng, (1024, 10))
    bn1, bn2 = wl.batchnorm_params(rng, 1024, K), wl.batchnorm_params(rng, 1024, 1024)
    thr1, flip1 = nets.fold(ctx, bn1, K)
    thr2, flip2 = nets.fold(ctx, bn2, 1024)
    W1p, W2p, W3p = (nets.pack_weight(ctx, W) for W in (W1, W2, W3))
    a1 = torch.empty(B, binding.packed_ld(1024), dtype=torch.int32, device="cuda")
    a2 = torch.empty_like(a1)
    S = torch.empty(B, 10, dtype=torch.int32, device="cuda")
    final = torch.empty(nets.convnet_output_shape(cnet, B, hw, hw), dtype=torch.int32, device="cuda")

    def full_net():
        ctx.convnet_forward(desc, Xc, B, hw, hw, final)
        ctx.binary_dense(final.view(B, K // 32), W1p, thr1, flip1, B, 1024, K, out=a1)
        ctx.binary_dense(a1, W2p, thr2, flip2, B, 1024, 1024, out=a2)
        ctx.xnor_gemm(a2, W3p, B, 10, 1024, C=S)
    ms = median_ms(full_net)
    out["convnet_with_fc_tail_8192_1024_1024_10_batch256"] = {"ms": ms, "images_per_s": B / (ms / 1e3)}
    ctx.set_workspace(None)
    return out


def bench_filter_repetition(ctx, median_ms, engine):
    """Section 3.3 on one layer (32 x 32 maps, 128 -> 128 channels, batch 64): how many 2-D filters are distinct, how many
    XNOR-popcount filter applications that leaves, and what the mechanism costs on this GPU next to the direct product on
    either engine.  iid weights (nearly every class occurs) and dictionary weights with 42 % distinct filters per channel,
    the share the paper reports for its trained CIFAR-10 network (trained weights are not available here)."""
    import torch
    from paper_1602_02830_b200 import workloads as wl
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    B, H, W, Cin, Cout = 64, 32, 32, 128, 128
    rng = np.random.default_rng(33)
    act = wl.pm1(rng, (B, H, W, Cin))
    actp = ctx.pack_signs(torch.from_numpy(act.reshape(B * H * W, Cin)).cuda()).view(B, H, W, -1)[..., :Cin // 32].contiguous()
    thr = torch.zeros(Cout, dtype=torch.int32, device="cuda")
    out = {"layer": "batch 64, 32 x 32, 128 -> 128 channels, no pooling", "filter_applications_direct": Cout * Cin,
           "note": "op counts are 2-D filter applications per output pixel (one XNOR-popcount on a 9-bit neighbourhood each); "
                   "the exploit adds C_out * C_in small-integer additions per pixel to combine the responses"}
    need = max(ctx.filter_repetition_workspace_bytes(Cin, Cout), ctx.conv_workspace_bytes(B, H, W, Cin, Cout, False), 256)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    ctx.set_workspace(ws)
    for name, wgt in (("iid_weights", wl.pm1(rng, (Cout, 3, 3, Cin))),
                      ("dictionary_42pct", wl.dictionary_conv_weights(rng, Cout, Cin, int(round(0.42 * Cout))))):
        flat = torch.from_numpy(wgt.reshape(Cout, 9 * Cin)).cuda()
        Wp = ctx.pack_signs(flat)[:, :9 * Cin // 32].contiguous()
        distinct = ctx.filter_repetition_count(Wp, Cin, Cout)
        row = {"distinct_2d_filters": distinct, "distinct_fraction": distinct / (Cout * Cin),
               "filter_applications_with_exploit": distinct, "reduction": (Cout * Cin) / distinct}
        ctx.set_conv_filter_repetition(True)
        row["exploit_ms"] = median_ms(lambda: ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, thr=thr), 5, 2)
        ctx.set_conv_filter_repetition(False)
        for ename, eng in (("direct_popc_ms", 1), ("direct_selected_engine_ms", engine)):
            ctx.set_engine(eng)
            row[ename] = median_ms(lambda: ctx.binary_conv2d(actp, B, H, W, Cin, Wp, Cout, thr=thr), 5, 2)
        ctx.set_engine(engine)
        out[name] = row
    out["verdict"] = ("the mechanism is exact but loses on this GPU: the direct product on the tensor cores (and on the CUDA-core "
                      "popcount kernel) is faster than applying even 42 % of the 2-D filters on CUDA cores")
    ctx.set_workspace(None)
    return out


if __name__ == "__main__":
    sys.exit(main())
