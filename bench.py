#!/usr/bin/env python
"""Benchmark of the ternary pointwise-convolution path.

One step = the 34 pointwise layers of MobileNetV2-1.0 at 224x224 for a batch of
128 images, chained through `prom_pw_layer_seq` (int8 NHWC activations,
2-bit ternary weights, fused requantisation).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...

`--impl reference` times the plain CPU oracle instead (host cores, bounded
sample per step).  `--single M,K,N[,variant]` times one layer.  `--sweep FILE` runs the shape/sparsity sweep of single
layers (tensor-core and add/sub variants) and writes one JSON record per point.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

BATCH = 128
METRIC = "MobileNetV2 all-1x1-layers images/s"
UNIT = "images/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
INT8_OVER_BF16 = 2.0          # nominal dense int8 : bf16 tensor ratio on B200 (4.5 : 2.25)
FLUSH_BYTES = 512 << 20       # > 2x the 126 MB L2
NCU_TRAFFIC_PER_LAUNCH = 15.46e6
NOMINAL_I8_TOPS = 4500.0      # data-sheet dense int8 figure of the part, for context


# --------------------------------------------------------------------------- helpers
def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    except Exception:
        return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS,
                    bf16_tflops_sustained=1400.0, source="fallback")


def layer_bytes(m, cin, cout):
    """Algorithmic bytes of one layer: activations in, activations out, 2-bit
    weights, 9 bytes of requantisation constants per output channel."""
    return m * cin + m * cout + cout * ((cin + 3) // 4) + 9 * cout


def layer_ops(m, cin, cout):
    return 2 * m * cin * cout


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU while a region runs."""

    def __init__(self, device_index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    _NAMES = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
              0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
              0x10: "sync_boost", 0x100: "display_clock_setting"}

    def _once(self):
        nv = self._nv
        mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
        try:
            r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
        except Exception:
            r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
        self.samples.append(mhz)
        for bit, name in self._NAMES.items():
            if r & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                return
            time.sleep(0.02)

    def start(self):
        if self._h is None:
            return
        self._stop.clear()
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def stop(self):
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
            self._thr = None

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def i8_peak_probe(torch, binding, iters=8192, reps=5, sustained_s=0.0):
    """Measured tensor-pipe rate on tcgen05.mma.kind::i8 (128x256x32, operands fixed in shared
    memory, one CTA per SM): the best of `reps` launches (burst) and, when asked, launches back to
    back for `sustained_s` seconds."""
    cycles = torch.zeros((4096,), dtype=torch.int64, device="cuda")
    grid = binding.debug_i8_mma_rate(256, cycles)
    torch.cuda.synchronize()
    ops_per_launch = grid * iters * 4 * 2 * 128 * 256 * 32
    stream = torch.cuda.current_stream()
    best = None
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        binding.debug_i8_mma_rate(iters, cycles)
        e1.record(stream)
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        best = ms if best is None or ms < best else best
    cyc = int(cycles[:grid].max().item())
    out = {"shape": "128x256x32 kind::i8, cta_group::1, one issuing thread per SM", "ctas": grid,
           "iters": iters, "tops_burst": ops_per_launch / best / 1e9,
           "macs_per_clk_per_sm": iters * 4 * 128 * 256 * 32 / cyc,
           "sm_mhz_from_cycles": cyc / best / 1e3}
    if sustained_s > 0:
        n = max(1, int(sustained_s * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            binding.debug_i8_mma_rate(iters, cycles)
        e1.record(stream)
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        out["tops_sustained"] = ops_per_launch * n / ms / 1e9
        out["sustained_s"] = ms / 1e3
    return out


def alu_rate_probe(torch, binding, iters=2000):
    """Measured issue rates (lanes per clock per SM) of the requantiser's 32-bit high multiply and,
    beside it, of mad.lo.s32, fma.rn.f32, mad.wide.s32, the saturating pack, a shift and fma.rn.f64:
    8 independent chains per thread, 1024 threads per SM."""
    cycles = torch.zeros((4096,), dtype=torch.int64, device="cuda")
    sink = torch.zeros((1,), dtype=torch.int32, device="cuda")
    out = {}
    for op, name in ((0, "mul_hi_s32"), (1, "mad_lo_s32"), (2, "fma_f32"), (3, "mad_wide_s32"),
                     (4, "cvt_pack_sat_u8"), (5, "shr_s32"), (6, "fma_f64")):
        binding.debug_alu_rate(op, 100, sink, cycles)
        grid = binding.debug_alu_rate(op, iters, sink, cycles)
        torch.cuda.synchronize()
        cyc = int(cycles[:grid].max().item())
        out[name] = round(1024 * 64 * iters / cyc, 2)
    return out


def write_bandwidth_probe(torch, gib=1):
    """What the GPU sustains when it only writes: a fill and a memset of `gib` GiB, best of 5 each
    (GB/s).  A copy moves read + write bytes at the copy bandwidth, i.e. half of it each way; a
    kernel that writes far more than it reads (an expand layer) is held to this figure instead."""
    n = gib << 30
    buf = torch.empty((n,), dtype=torch.uint8, device="cuda")
    out = {}
    for name, fn in (("fill", lambda: buf.fill_(3)), ("memset", lambda: buf.zero_())):
        ts = []
        for i in range(7):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            if i >= 2:
                ts.append(e0.elapsed_time(e1))
        out[name + "_gbs"] = round(n / min(ts) / 1e6, 1)
    del buf
    out["gbs"] = max(out["fill_gbs"], out["memset_gbs"])
    out["how"] = f"torch fill_ / zero_ over {gib} GiB of uint8, best of 5, CUDA events"
    return out


def mma_issue_probe(torch, binding, iters=4096):
    """SM clocks per tcgen05.mma.kind::i8 of shape 128 x N x 32, per SM and per issuing thread, for
    1, 2 and 4 issuing threads (as far as tensor memory holds their accumulators)."""
    cycles = torch.zeros((4096,), dtype=torch.int64, device="cuda")
    out = []
    for n in (16, 32, 64, 128, 256):
        for warps in (1, 2, 4):
            if warps * 2 * max(n, 64) > 512:
                continue
            binding.debug_mma_issue_rate(n, warps, 64, cycles)
            grid = binding.debug_mma_issue_rate(n, warps, iters, cycles)
            torch.cuda.synchronize()
            cyc = int(cycles[:4 * grid].max().item())
            out.append({"n": n, "issuing_threads": warps, "cycles_per_mma_per_sm": round(cyc / (4.0 * iters * warps), 1),
                        "cycles_per_mma_per_thread": round(cyc / (4.0 * iters), 1)})
    return out


def l2_copy_probe(torch, binding, iters=4096, region_mb=8):
    """Bytes per SM clock that every SM pulls from an L2-resident region with 16 KB bulk copies,
    against the number of copies it keeps in flight; and the total in TB/s by CUDA events."""
    cycles = torch.zeros((1024,), dtype=torch.int64, device="cuda")
    region = torch.ones((region_mb << 20,), dtype=torch.uint8, device="cuda")
    out = []
    for stages in (1, 2, 3, 4, 6, 8):
        binding.debug_l2_copy_rate(region, 256, stages, cycles)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        grid = binding.debug_l2_copy_rate(region, iters, stages, cycles)
        e1.record()
        e1.synchronize()
        cyc = int(cycles[:grid].max().item())
        out.append({"copies_in_flight": stages, "bytes_per_clk_per_sm": round(iters * 16384 / cyc, 1),
                    "tb_per_s_all_sms": round(iters * 16384 * grid / (e0.elapsed_time(e1) * 1e-3) / 1e12, 2)})
    return out


def mma_beside_probe(torch, binding, iters=4096):
    """128 x 128 x 32 MMAs beside bulk copies into the same SM's shared memory, and beside warps that
    read tensor memory: SM clocks per MMA, bytes per clock of the copies, bytes per clock of the reads."""
    out = torch.zeros((8 * 1024,), dtype=torch.int64, device="cuda")
    region = torch.ones((8 << 20,), dtype=torch.uint8, device="cuda")
    rows = {"beside_copies": [], "beside_reads": []}
    for stages in (0, 1, 2, 3):
        binding.debug_mma_beside(0, 64, 0, stages, region, out)
        grid = binding.debug_mma_beside(0, iters, 0, stages, region, out)
        torch.cuda.synchronize()
        o = out[:8 * grid].view(grid, 8)
        cyc = int(o[:, 0].max().item())
        rows["beside_copies"].append({"copies_in_flight": stages, "cycles_per_mma": round(cyc / (4.0 * iters), 1),
                                      "copy_bytes_per_clk_per_sm": round(float(o[:, 3].double().mean().item()) * 16384 / cyc, 1)})
    for nwarps in (4, 8, 16):
        for mma in (0, 1):
            binding.debug_mma_beside(1, 64, nwarps, mma, None, out)
            grid = binding.debug_mma_beside(1, iters, nwarps, mma, None, out)
            torch.cuda.synchronize()
            o = out[:8 * grid].view(grid, 8)
            cyc = int(o[:, 0].max().item())
            n_mma = o[:, 1].double()
            c_mma = o[:, 2].double()
            rows["beside_reads"].append({"reading_warps": nwarps, "mmas": bool(mma),
                                         "read_bytes_per_clk_per_sm": round(iters * nwarps * 4096.0 / cyc, 1),
                                         "cycles_per_mma": round(float((c_mma / n_mma.clamp(min=1)).max().item()), 1) if mma else None})
    return rows


def build_network(seed, synth, binding=None, device=None, width=1.0):
    """Layer table plus per-layer weights/constants: host arrays for the oracle,
    and (when a binding is given) packed device tensors for the library."""
    table = synth.mobilenetv2_pointwise_layers(width=width)
    host, dev = [], []
    for i, l in enumerate(table):
        d = synth.make_layer(seed, l.cin, l.cout, 0.5, index=i + 1)
        host.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w=d["w"].numpy(),
                         bias=d["bias"].numpy(), mult=d["mult"].numpy(), shift=d["shift"].numpy()))
        if binding is not None:
            dev.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride,
                            w_packed=binding.pack_ternary(d["w"].to(device)),
                            bias=d["bias"].to(device), mult=d["mult"].to(device),
                            shift=d["shift"].to(device)))
    return table, host, dev


# --------------------------------------------------------------------------- reference arm
def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step is the whole
    34-layer sequence over a bounded number of images."""
    rank, _, _ = rank_info()
    if rank != 0:
        return 0
    from oracle import prom_oracle
    from paper_2505_03254_b200 import synth
    prom_oracle.build()
    seed = synth.BASE_SEED + 3
    _, host, _ = build_network(seed, synth)
    x1 = synth.act_post_relu6(seed, (1, 112, 112, 32)).numpy()
    t0 = time.perf_counter()
    prom_oracle.layer_seq(host, x1)
    t1 = max(time.perf_counter() - t0, 1e-4)
    total = args.steps + args.warmup
    images = int(max(1, min(BATCH, 120.0 / (total * t1))))
    x = synth.act_post_relu6(seed, (images, 112, 112, 32)).numpy()
    for _ in range(args.warmup):
        prom_oracle.layer_seq(host, x)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        prom_oracle.layer_seq(host, x)
    dt = time.perf_counter() - t0
    value = images * args.steps / dt
    cores = prom_oracle.threads()
    sample = f"{images} image(s) of the batch-{BATCH} workload per step, all 34 layers"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "configs[2]: MobileNetV2-1.0 @224, all 34 1x1 layers, chained, "
                               f"batch {BATCH}; reference arm steps over {images} image(s)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)
    return 0


# --------------------------------------------------------------------------- ranks
def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(ms, device="cuda"):
    """The slowest rank's time: every multi-GPU number is the max over ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(images_per_rank_per_step, steps, world, ms):
    """Aggregate images/s of the job: all ranks' images over the slowest rank's time."""
    return world * images_per_rank_per_step * steps / (ms * 1e-3)


def spawn_ranks(args, argv):
    """`--gpus N` without a launcher's environment: start N ranks of this script itself, one
    process per GPU (LOCAL_RANK picks the device), rendezvous on 127.0.0.1.  Rank 0 prints the
    JSON line; the exit code is the worst of the ranks'."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env))
    rc = 0
    for pr in procs:
        rc = max(rc, abs(pr.wait()))
    return rc


def run_stub(args):
    """The multi-rank bookkeeping of the GPU arm with the step replaced by a fixed per-rank time
    and `gloo` in place of NCCL: what a machine without GPUs can run of `--gpus N`."""
    import torch.distributed as dist
    rank, _, world = rank_info()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo", rank=rank, world_size=world)
        dist.barrier()
    ms = max_over_ranks(10.0 + 5.0 * rank, device="cpu")
    if rank == 0:
        print(json.dumps({"impl": "stub", "metric": METRIC, "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "ms_per_step": ms / args.steps,
                          "value": whole_job_value(BATCH, args.steps, world, ms), "scaling": "weak"}),
              flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


# --------------------------------------------------------------------------- GPU arm
def time_region(torch, fn, steps, dist_on):
    """Times `steps` calls of fn with CUDA events on the current stream, bracketed
    by barrier + synchronize; returns milliseconds (max over ranks)."""
    import torch.distributed as dist
    stream = torch.cuda.current_stream()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    if dist_on:
        dist.barrier()
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    if dist_on:
        dist.barrier()
    return max_over_ranks(e0.elapsed_time(e1))


def cold_time_us(torch, fn, flush, iters=20, warm=3):
    """Median/min device time of one launch with L2 flushed before each."""
    stream = torch.cuda.current_stream()
    ts = []
    for i in range(warm + iters):
        flush.fill_(i & 0x7F)
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        e1.synchronize()
        if i >= warm:
            ts.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(ts), min(ts)


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2505_03254_b200 import binding, build, synth

    rank, local, world = rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dist_on = world > 1
    if dist_on:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if dist_on:
        dist.barrier()
    binding.lib()
    pk = peaks()
    bw = pk["hbm_gbs"] * 1e9

    seed = synth.BASE_SEED + 3
    table, host, dev = build_network(seed, synth, binding, "cuda")
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(seed, (BATCH, 112, 112, 32), device="cuda")
    ws = torch.empty((seq.workspace_bytes(BATCH, 112, 112),), dtype=torch.uint8, device="cuda")
    y = torch.empty((BATCH, 7, 7, 1280), dtype=torch.int8, device="cuda")
    variant = args.variant

    side = torch.cuda.Stream()

    def step_plain():
        binding.pw_layer_seq(seq, x0, ws, y_out=y, variant=variant)

    l0 = binding.launch_count()
    step_plain()
    launches_per_step = binding.launch_count() - l0
    torch.cuda.synchronize()
    graph = None
    if not args.no_graph:
        # the step's launches (one prep kernel + one kernel per layer) captured once and replayed
        with torch.cuda.stream(side):
            binding.pw_layer_seq(seq, x0, ws, y_out=y, variant=variant, stream=side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            binding.pw_layer_seq(seq, x0, ws, y_out=y, variant=variant, stream=side)
    step = graph.replay if graph is not None else step_plain

    sampler = ClockSampler(local)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if binding.last_device_status() != binding.PROM_OK:
        raise RuntimeError("device status not OK after warm-up")

    # ---- device-resident timing ------------------------------------------------
    sampler.start()
    ms = time_region(torch, step, args.steps, dist_on)
    launches = launches_per_step * args.steps
    ms_per_step = ms / args.steps
    value = whole_job_value(BATCH, args.steps, world, ms)
    ms_plain = time_region(torch, step_plain, min(args.steps, 200), dist_on) / min(args.steps, 200)

    # ---- end to end: pinned host input -> device -> sequence -> host output ------
    x0_host = x0.cpu().pin_memory()
    y_host = torch.empty((BATCH, 7, 7, 1280), dtype=torch.int8).pin_memory()
    ws_host = torch.empty((seq.host_workspace_bytes(BATCH, 112, 112),), dtype=torch.uint8,
                          device="cuda")

    def step_e2e():
        binding.pw_layer_seq_host(seq, x0_host, ws_host, y_host, variant=variant)

    for _ in range(3):
        step_e2e()
    e2e_steps = args.steps
    ms_e2e_serial = time_region(torch, step_e2e, e2e_steps, dist_on)
    same = bool(torch.equal(y_host, y.cpu()))

    # The same call issued alternately on two streams, each with its own workspace and pinned
    # output: the copies of one step overlap the kernels of the other (every step still copies
    # its input in and its result out).
    lanes = []
    for _ in range(2):
        lanes.append(dict(st=torch.cuda.Stream(), ws=torch.empty_like(ws_host),
                          y=torch.empty_like(y_host).pin_memory(), ev=torch.cuda.Event()))
    turn = [0]

    def step_e2e_pipelined():
        ln = lanes[turn[0] & 1]
        turn[0] += 1
        binding.pw_layer_seq_host(seq, x0_host, ln["ws"], ln["y"], variant=variant, stream=ln["st"])

    def fork():
        ev = torch.cuda.Event()
        ev.record(torch.cuda.current_stream())
        for ln in lanes:
            ln["st"].wait_event(ev)

    def join():
        for ln in lanes:
            ln["ev"].record(ln["st"])
            torch.cuda.current_stream().wait_event(ln["ev"])

    def region_pipelined():
        fork()
        for _ in range(e2e_steps):
            step_e2e_pipelined()
        join()

    fork()
    for _ in range(4):
        step_e2e_pipelined()
    join()
    torch.cuda.synchronize()
    ms_e2e = time_region(torch, region_pipelined, 1, dist_on)
    sampler.stop()
    same = same and all(bool(torch.equal(ln["y"], y_host)) for ln in lanes)
    if ms_e2e > ms_e2e_serial:          # never report the slower of the two ways to call it
        ms_e2e = ms_e2e_serial
    e2e_value = whole_job_value(BATCH, e2e_steps, world, ms_e2e)
    del ws_host, lanes

    status = binding.last_device_status()
    if status != binding.PROM_OK:
        raise RuntimeError(f"device status {status} after the timed region")

    # the tensor and integer-multiply roofs are measured here, on this GPU, once the timed
    # regions are over (the probes draw full power; nothing is timed in their wake)
    i8 = i8_peak_probe(torch, binding, sustained_s=0.25)
    alu = alu_rate_probe(torch, binding)
    p_i8 = i8["tops_burst"] * 1e12
    torch.cuda.synchronize()
    time.sleep(0.5)

    # ---- roofline of the step ----------------------------------------------------
    ms_layers = [BATCH * l.h * l.w for l in table]
    step_bytes = sum(layer_bytes(m, l.cin, l.cout) for m, l in zip(ms_layers, table))
    step_ops = sum(layer_ops(m, l.cin, l.cout) for m, l in zip(ms_layers, table))
    roof_us = [max(layer_bytes(m, l.cin, l.cout) / bw, layer_ops(m, l.cin, l.cout) / p_i8) * 1e6
               for m, l in zip(ms_layers, table)]
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "tc_conv_kernel", "achieved": achieved,
                "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"],
                "peak_source": pk["source"],
                # dram read + write bytes per tc_conv_kernel launch (average over the step's 34
                # launches) from the ncu capture summarised in profiles/; None once the kernel changes
                "traffic": NCU_TRAFFIC_PER_LAUNCH,
                "launches_per_step": launches / args.steps,
                "bytes_per_launch": step_bytes / (launches / args.steps),
                "us_per_launch": ms_per_step * 1e3 / (launches / args.steps),
                "step_roofline_us": sum(roof_us),
                "step_roofline_frac": sum(roof_us) / (ms_per_step * 1e3)}

    # The copy bandwidth is read + write; on its own the write path sustains less than the copy's
    # total (measured here), and the expand layers write six times what they read.  Beside the
    # figure against the copy bandwidth, the step's roofline with the write path as a third roof.
    if rank == 0:
        wr = write_bandwidth_probe(torch)
        roof_w_us = [max(r, m * l.cout / (wr["gbs"] * 1e9) * 1e6) for r, m, l in zip(roof_us, ms_layers, table)]
        roofline["write_path"] = {"gbs": wr["gbs"], "probe": wr, "step_roofline_us": sum(roof_w_us),
                                  "step_roofline_frac": sum(roof_w_us) / (ms_per_step * 1e3),
                                  "layers_bound_by_it": sum(1 for a, b in zip(roof_w_us, roof_us) if a > b)}

    # second roof of the requantising epilogue: one 32-bit high multiply per output, at the rate
    # the probe above measured on this GPU (lanes per clock per SM) and the sampled SM clock
    step_outputs = sum(m * l.cout for m, l in zip(ms_layers, table))
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    clk = (sampler.summary()["sm_mhz"] or 1965) * 1e6
    alu_peak = sms * alu["mul_hi_s32"] * clk
    roofline["epilogue_alu"] = {"bound": "alu", "achieved": step_outputs / (ms_per_step * 1e-3),
                                "peak": alu_peak, "unit": "outputs/s",
                                "frac": step_outputs / (ms_per_step * 1e-3) / alu_peak,
                                "lanes_per_clk_per_sm": alu}
    # the tensor roof behind the compute-bound layers' figures: measured, with the two other
    # candidates beside it
    roofline["tensor_peak"] = {"used_tops": p_i8 / 1e12, "source": "measured here (tcgen05.mma.kind::i8 issue loop)",
                               "probe": i8, "two_x_measured_bf16_tops": INT8_OVER_BF16 * pk["bf16_tflops"],
                               "nominal_tops": NOMINAL_I8_TOPS,
                               "step_roofline_us_at_2x_bf16": sum(
                                   max(layer_bytes(m, l.cin, l.cout) / bw,
                                       layer_ops(m, l.cin, l.cout) / (INT8_OVER_BF16 * pk["bf16_tflops"] * 1e12)) * 1e6
                                   for m, l in zip(ms_layers, table)),
                               "step_roofline_us_at_nominal": sum(
                                   max(layer_bytes(m, l.cin, l.cout) / bw,
                                       layer_ops(m, l.cin, l.cout) / (NOMINAL_I8_TOPS * 1e12)) * 1e6
                                   for m, l in zip(ms_layers, table))}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": f"configs[2]: MobileNetV2-1.0 @224, all 34 ternary 1x1 layers, "
                               f"chained, batch {BATCH} per GPU, post-ReLU6 int8 NHWC input "
                               f"[{BATCH},112,112,32], P(0)=0.5 ternary weights",
                   "variant": variant, "seed": seed,
                   "launch": ("CUDA graph of the step's kernels, replayed" if graph is not None
                              else "plain launches"),
                   "l2": "no flush: a step moves 877 MB through buffers of up to 154 MB (> 126 MB L2)",
                   "parallelism": f"batch sharded over {world} GPU(s), no collective"},
        "gops": step_ops / (ms_per_step * 1e-3) / 1e9,
        "ms_per_step_plain_launches": ms_plain,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x0_host.numel()),
                "d2h_bytes_per_step": int(y_host.numel()), "ms_per_step": ms_e2e / e2e_steps,
                "ms_per_step_one_stream": ms_e2e_serial / e2e_steps,
                "how": "prom_pw_layer_seq_host on two streams alternately (two workspaces)",
                "matches_device_run": same},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "clocks": sampler.summary(),
    }

    if rank == 0 and world == 1 and not args.no_detail:
        out["layers"] = per_layer_detail(torch, binding, synth, table, dev, seed, bw, p_i8, variant)
        out["single_layer"] = single_layer_configs(torch, binding, synth, bw, p_i8)
        out["quantizer"] = quantizer_timing(torch, binding, table, bw)
        out["act_quantizer"] = act_quantizer_timing(torch, binding, bw)
        out["dynamic_layer"] = dynamic_layer_timing(torch, binding, synth, bw)
        out["depthwise"] = depthwise_timing(torch, binding, bw)
        out["body_with_depthwise"] = body_with_depthwise_timing(torch, binding, synth, bw)
        out["body_with_skip_connections"] = body_with_depthwise_timing(torch, binding, synth, bw, skips=True)
        cold_us = sum(r["us"] for r in out["layers"])
        roofline["sum_layer_cold_us"] = cold_us
        roofline["sum_layer_cold_frac"] = sum(roof_us) / cold_us

    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle import prom_oracle
        prom_oracle.build()
        xh = x0_host.numpy()
        t0 = time.perf_counter()
        want = prom_oracle.layer_seq(host, xh)
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": BATCH / dt, "unit": UNIT, "cores": prom_oracle.threads(),
                               "kind": "oracle",
                               "sample": f"one full step (batch {BATCH}, 34 layers), {dt:.2f} s"}
        out["parity"] = bool((want == y.cpu().numpy()).all())
    elif rank == 0:
        out["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist_on:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def per_layer_detail(torch, binding, synth, table, dev, seed, bw, p_i8, variant):
    """Cold-L2 time of every layer on its own (a one-layer sequence so that the
    stride-2 sampling stays folded into the loads)."""
    flush = torch.empty((FLUSH_BYTES,), dtype=torch.uint8, device="cuda")
    rows = []
    for i, (l, d) in enumerate(zip(table, dev)):
        hin, win = l.h * l.in_stride, l.w * l.in_stride
        x = synth.act_post_relu6(seed + 100 + i, (BATCH, hin, win, l.cin), device="cuda")
        yy = torch.empty((BATCH, l.h, l.w, l.cout), dtype=torch.int8, device="cuda")
        one = binding.LayerSeq([d])
        wsd = torch.empty((16,), dtype=torch.uint8, device="cuda")
        fn = lambda: binding.pw_layer_seq(one, x, wsd, y_out=yy, variant=variant)
        med, mn = cold_time_us(torch, fn, flush)
        m = BATCH * l.h * l.w
        b, o = layer_bytes(m, l.cin, l.cout), layer_ops(m, l.cin, l.cout)
        roof = max(b / bw, o / p_i8) * 1e6
        rows.append({"i": i + 1, "name": l.name, "k": l.cin, "n": l.cout, "m": m,
                     "stride": l.in_stride, "us": round(med, 2), "us_min": round(mn, 2),
                     "gbs": round(b / med / 1e3, 1), "tops": round(o / med / 1e6, 1),
                     "roof_us": round(roof, 2), "frac": round(roof / med, 3)})
        del x, yy
    return rows


def quantizer_timing(torch, binding, table, bw):
    """The step before the path (off the timed step): float weights of all 34 layers ->
    alpha and 2-bit ternary codes, one launch per layer, L2 flushed before the batch."""
    import math
    g = torch.Generator(device="cuda").manual_seed(1)
    ws = [torch.randn((l.cout, l.cin), generator=g, device="cuda") * math.sqrt(2.0 / l.cout) for l in table]
    flush = torch.empty((FLUSH_BYTES,), dtype=torch.uint8, device="cuda")
    jobs = binding.QuantizeJobs(ws)                     # marshalled once: the call itself is what is timed
    binding.quantize_ternary_batch(jobs=jobs)
    fn = lambda: binding.quantize_ternary_batch(jobs=jobs)
    med, mn = cold_time_us(torch, fn, flush, iters=10)
    fn_each = lambda: [binding.quantize_ternary(w) for w in ws]
    med_each, _ = cold_time_us(torch, fn_each, flush, iters=5)
    nbytes = sum(4 * w.numel() + (w.shape[0] * ((w.shape[1] + 3) // 4)) + 4 * w.shape[0] for w in ws)
    return {"workload": "float32 weights of the 34 layers (2.1 M) -> alpha + 2-bit codes, one launch",
            "us": round(med, 2), "us_min": round(mn, 2), "us_one_launch_per_layer": round(med_each, 2), "bytes": nbytes,
            "gbs": round(nbytes / med / 1e3, 1), "roof_us": round(nbytes / bw * 1e6, 2),
            "frac": round(nbytes / bw * 1e6 / med, 4)}


def act_quantizer_timing(torch, binding, bw):
    """The step after the path in the paper's dataflow (off the timed step): per-sample absmax
    quantisation of a float32 activation tensor of the first layer's input shape
    [128,112,112,32] (205 MB > L2) to int8.  Algorithmic bytes: 4 read + 1 written per value."""
    g = torch.Generator(device="cuda").manual_seed(2)
    x = torch.randn((BATCH, 112, 112, 32), generator=g, device="cuda")
    out = (torch.empty(x.shape, dtype=torch.int8, device="cuda"),
           torch.empty((BATCH,), dtype=torch.float32, device="cuda"),
           torch.empty((BATCH,), dtype=torch.float32, device="cuda"))
    fn = lambda: binding.quantize_act_absmax(x, out=out)
    for _ in range(3):
        fn()
    ms = time_region(torch, fn, 20, False) / 20
    nbytes = 5 * x.numel() + 8 * BATCH
    return {"workload": "float32 [128,112,112,32] -> int8 + per-sample gamma and scale, one launch",
            "us": round(ms * 1e3, 2), "bytes": nbytes, "gbs": round(nbytes / ms / 1e6, 1),
            "roof_us": round(nbytes / bw * 1e6, 2), "frac": round(nbytes / bw * 1e3 / ms, 4)}


def dynamic_layer_timing(torch, binding, synth, bw):
    """The widest layer of the step (1 605 632 x 16 -> 96, 128 samples) in the paper's dynamic
    form (prom_pw_conv_i8_dyn: two tensor-core passes, per-sample scales), off the timed step.
    Algorithmic bytes: the input read twice, the output written once, nothing else."""
    batch, rows, k, n = BATCH, 112 * 112, 16, 96
    m = batch * rows
    x = synth.act_uniform_i8(synth.BASE_SEED + 40, (m, k), device="cuda")
    lay = synth.make_layer(synth.BASE_SEED + 40, k, n, 0.5, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    g = torch.Generator(device="cuda").manual_seed(3)
    alpha = torch.rand((n,), generator=g, device="cuda") * 0.1 + 0.01
    gx = torch.rand((batch,), generator=g, device="cuda") * 4 + 0.5
    out = (torch.empty((m, n), dtype=torch.int8, device="cuda"),
           torch.empty((batch,), dtype=torch.float32, device="cuda"),
           torch.empty((batch,), dtype=torch.float32, device="cuda"))
    fn = lambda: binding.pw_conv_i8_dyn(x, batch, wp, n, alpha, gx, out=out)
    for _ in range(3):
        fn()
    ms = time_region(torch, fn, 20, False) / 20
    nbytes = 2 * m * k + m * n
    return {"workload": "1605632x16->96, 128 samples: convolution, dequantise, per-sample absmax, quantise",
            "us": round(ms * 1e3, 2), "bytes": nbytes, "gbs": round(nbytes / ms / 1e6, 1),
            "roof_us": round(nbytes / bw * 1e6, 2), "frac": round(nbytes / bw * 1e3 / ms, 4)}


def depthwise_timing(torch, binding, bw):
    """The int8 depthwise 3x3 convolutions of the first blocks at batch 128 (off the timed step,
    where the depthwise layer is an identity stand-in): the two largest of the network."""
    g = torch.Generator(device="cuda").manual_seed(4)
    rows = []
    for (h, c, s) in ((112, 96, 2), (56, 144, 1)):
        x = torch.randint(-128, 128, (BATCH, h, h, c), generator=g, device="cuda", dtype=torch.int8)
        w = torch.randint(-128, 128, (c, 3, 3), generator=g, device="cuda", dtype=torch.int8)
        bias = torch.zeros((c,), dtype=torch.int32, device="cuda")
        rq = binding.make_requant(bias, bias + (1 << 30), torch.full((c,), 8, dtype=torch.int8, device="cuda"))
        ho = (h - 1) // s + 1
        y = torch.empty((BATCH, ho, ho, c), dtype=torch.int8, device="cuda")
        fn = lambda: binding.dw_conv3x3_i8(x, w, rq, stride=s, y=y)
        for _ in range(3):
            fn()
        ms = time_region(torch, fn, 20, False) / 20
        nbytes = x.numel() + y.numel()
        rows.append({"shape": "[%d,%d,%d,%d] stride %d" % (BATCH, h, h, c, s), "us": round(ms * 1e3, 2),
                     "gbs": round(nbytes / ms / 1e6, 1), "roof_us": round(nbytes / bw * 1e6, 2),
                     "frac": round(nbytes / bw * 1e3 / ms, 4)})
    return rows


def body_with_depthwise_timing(torch, binding, synth, bw, skips=False):
    """The 34 pointwise layers with a real int8 depthwise 3x3 in front of every project
    convolution (17 of them) in place of the identity stand-in: the body of MobileNetV2, batch
    128, CUDA graph.  With `skips` the project layers are linear (clamp [-128, 127]) and the ten
    blocks that keep their input's shape add it to their output in the project layer's epilogue.
    Algorithmic bytes: the pointwise layers' plus one byte in and one byte out per depthwise
    value, plus one byte per output of a block with a skip connection."""
    seed = synth.BASE_SEED + 3
    table, _, dev = build_network(seed, synth, binding, "cuda")
    g = torch.Generator(device="cuda").manual_seed(5)
    nbytes = 0
    for l, d in zip(table, dev):
        m = BATCH * l.h * l.w
        nbytes += layer_bytes(m, l.cin, l.cout)
        if l.name.endswith("project"):
            c = l.cin
            d["dw_w"] = torch.randint(-20, 21, (c, 3, 3), generator=g, device="cuda", dtype=torch.int8)
            d["dw_bias"] = torch.zeros((c,), dtype=torch.int32, device="cuda")
            d["dw_mult"] = torch.full((c,), 1 << 30, dtype=torch.int32, device="cuda")
            d["dw_shift"] = torch.full((c,), 6, dtype=torch.int8, device="cuda")
            nbytes += m * c * l.in_stride * l.in_stride + m * c
            if skips:
                d["act_min"] = -128
    n_skips = 0
    if skips:
        for i, (l, d) in enumerate(zip(table, dev)):
            if synth.has_skip_connection(table, i):
                d["add_block_input"] = True
                nbytes += BATCH * l.h * l.w * l.cout
                n_skips += 1
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(seed, (BATCH, 112, 112, 32), device="cuda")
    ws = torch.empty((seq.workspace_bytes(BATCH, 112, 112),), dtype=torch.uint8, device="cuda")
    y = torch.empty((BATCH, 7, 7, 1280), dtype=torch.int8, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()          # the inputs were made on the default stream
    with torch.cuda.stream(side):
        binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
    for _ in range(3):
        graph.replay()
    ms = time_region(torch, graph.replay, 50, False) / 50
    return {"workload": "34 pointwise + 17 depthwise 3x3 layers, chained, batch 128"
                        + (f", linear project layers, {n_skips} skip connections" if skips else ""),
            "ms_per_step": round(ms, 4), "images_per_s": round(BATCH / ms * 1e3, 1), "bytes": nbytes,
            "roof_us": round(nbytes / bw * 1e6, 1), "frac": round(nbytes / bw * 1e3 / ms, 4),
            "device_status": binding.last_device_status()}


def depth_first_timing(torch, binding, synth):
    """The three runs of late layers of the network (28x28, 14x14 and 7x7 feature maps) and the
    whole step, each as a CUDA graph, with one launch per layer, with the depth-first launches
    of prom_debug_seq_chain(1) and with the runs that stay in shared memory of
    prom_debug_seq_chain(2); outputs compared."""
    table = synth.mobilenetv2_pointwise_layers()
    seed = synth.BASE_SEED + 3
    rows = []
    for lo, hi in ((6, 12), (12, 26), (26, 34), (0, 34)):
        res = {}
        outs = []
        for mode in (0, 1, 2):
            binding.debug_seq_chain(mode)
            dev = []
            for i, l in enumerate(table[lo:hi]):
                d = synth.make_layer(seed, l.cin, l.cout, 0.5, index=lo + i + 1, device="cuda")
                dev.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w_packed=binding.pack_ternary(d["w"]),
                                bias=d["bias"], mult=d["mult"], shift=d["shift"]))
            seq = binding.LayerSeq(dev)
            l0, ll = table[lo], table[hi - 1]
            hin, win = l0.h * l0.in_stride, l0.w * l0.in_stride
            x0 = synth.act_post_relu6(seed, (BATCH, hin, win, l0.cin), device="cuda")
            ws = torch.empty((max(16, seq.workspace_bytes(BATCH, hin, win)),), dtype=torch.uint8, device="cuda")
            y = torch.empty((BATCH, ll.h, ll.w, ll.cout), dtype=torch.int8, device="cuda")
            side = torch.cuda.Stream()
            torch.cuda.synchronize()          # the inputs were made on the default stream
            with torch.cuda.stream(side):
                binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
            for _ in range(5):
                g.replay()
            res[mode] = time_region(torch, g.replay, 200, False) / 200 * 1e3
            outs.append(y.clone())
            res[("status", mode)] = binding.last_device_status()
        binding.debug_seq_chain(0)
        rows.append({"layers": f"{lo + 1}..{hi}", "us_one_launch_per_layer": round(res[0], 1),
                     "us_depth_first": round(res[1], 1), "us_resident_runs": round(res[2], 1),
                     "same_output": bool(torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])),
                     "device_status": [res[("status", m)] for m in (0, 1, 2)]})
    return rows


def single_layer_configs(torch, binding, synth, bw, p_i8):
    """Configs 1, 2 and 4 as single layers (cold L2), every variant that runs them."""
    flush = torch.empty((FLUSH_BYTES,), dtype=torch.uint8, device="cuda")
    cases = [("configs[0]", 196, 64, 384, "i8"), ("configs[1]", 64 * 112 * 112, 16, 96, "relu6"),
             ("configs[3]a", 25088, 960, 160, "u7"), ("configs[3]b", 25088, 160, 960, "u7"),
             ("configs[3]c", 25088, 320, 1280, "u7")]
    out = []
    for ci, (name, m, cin, cout, act) in enumerate(cases):
        seed = synth.BASE_SEED + 10 + ci
        gen = {"i8": synth.act_uniform_i8, "relu6": synth.act_post_relu6,
               "u7": synth.act_uniform_0_127}[act]
        x = gen(seed, (m, cin), device="cuda")
        lay = synth.make_layer(seed, cin, cout, 0.5, device="cuda")
        wp = binding.pack_ternary(lay["w"])
        rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
        y = torch.empty((m, cout), dtype=torch.int8, device="cuda")
        b, o = layer_bytes(m, cin, cout), layer_ops(m, cin, cout)
        roof = max(b / bw, o / p_i8) * 1e6
        prep = binding.pw_prepare(m, cin, wp, cout, rq)
        for variant in ("tc", "tc_prepared", "addsub"):
            try:
                if variant == "tc_prepared":
                    if prep is None:
                        continue
                    fn = lambda: binding.pw_conv_i8_prepared(x, cout, prep, y=y)
                else:
                    fn = lambda: binding.pw_conv_i8(x, wp, cout, rq, y=y, variant=variant)
                fn()
            except binding.PromError:
                continue
            med, mn = cold_time_us(torch, fn, flush, iters=10 if variant == "addsub" else 20)
            out.append({"workload": name, "m": m, "k": cin, "n": cout, "variant": variant,
                        "us": round(med, 2), "gops": round(o / med / 1e3, 1),
                        "gbs": round(b / med / 1e3, 1), "roof_us": round(roof, 2),
                        "frac": round(roof / med, 4)})
    return out


# --------------------------------------------------------------------------- sweep
def sweep_rows(m, torch, tile=128, edge=512, one_in=64):
    """Rows the oracle checks at a sweep point: all of them up to 16384 rows, else the first and
    last `edge`, both rows at every tile boundary, and every `one_in`-th of the rest (staggered)."""
    if m <= 16384:
        return torch.arange(m, dtype=torch.int64)
    keep = torch.zeros(m, dtype=torch.bool)
    keep[:edge] = True
    keep[m - edge:] = True
    b = torch.arange(tile, m, tile, dtype=torch.int64)
    keep[b] = True
    keep[b - 1] = True
    keep[torch.arange(37, m, one_in + 1, dtype=torch.int64)] = True
    return torch.nonzero(keep).flatten()


def run_sweep(args):
    """Shape and sparsity sweep of single layers: the tensor-core variant (or what AUTO picks
    where it refuses the shape, labelled) and the add/sub variant on every point, each timed with
    a cold L2 and checked: the whole output against the plain one-thread-per-output kernel, and
    sampled rows against the CPU oracle."""
    import torch
    from paper_2505_03254_b200 import binding, build, synth
    torch.cuda.set_device(0)
    build.build()
    binding.lib()
    oracle = None
    if not args.no_cpu:
        from oracle import prom_oracle as oracle
        oracle.build()
    pk = peaks()
    i8 = i8_peak_probe(torch, binding)
    bw, p_i8 = pk["hbm_gbs"] * 1e9, i8["tops_burst"] * 1e12
    flush = torch.empty((FLUSH_BYTES,), dtype=torch.uint8, device="cuda")
    ms_list = synth.CONFIG5_M if not args.sweep_small else synth.CONFIG5_M[:2]
    n = bad = 0
    with open(args.sweep, "w") as f:
        f.write(json.dumps({"int8_peak_probe": i8, "hbm_gbs": pk["hbm_gbs"], "peak_source": pk["source"]}) + "\n")
        for m in ms_list:
            rows = sweep_rows(m, torch)
            rows_d = rows.cuda()
            for cin in synth.CONFIG5_CIN:
                x = synth.act_uniform_i8(synth.BASE_SEED + 5, (m, cin), device="cuda")
                x_rows = x[rows_d].cpu().numpy() if oracle is not None else None
                for cout in synth.CONFIG5_COUT:
                    y = torch.empty((m, cout), dtype=torch.int8, device="cuda")
                    y_ref = torch.empty((m, cout), dtype=torch.int8, device="cuda")
                    for z in synth.CONFIG5_ZERO:
                        lay = synth.make_layer(synth.BASE_SEED + 5, cin, cout, z, device="cuda")
                        wp = binding.pack_ternary(lay["w"])
                        rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
                        b, o = layer_bytes(m, cin, cout), layer_ops(m, cin, cout)
                        roof = max(b / bw, o / p_i8) * 1e6
                        nnz = int((lay["w"] != 0).sum().item())
                        binding.pw_conv_i8(x, wp, cout, rq, y=y_ref, variant="naive")
                        want, naive_ok = None, True
                        if oracle is not None:
                            want = torch.from_numpy(oracle.conv_mul(
                                x_rows, lay["w"].cpu().numpy(), lay["bias"].cpu().numpy(),
                                lay["mult"].cpu().numpy(), lay["shift"].cpu().numpy())).cuda()
                            naive_ok = bool(torch.equal(y_ref[rows_d], want))
                        for variant in ("tc", "addsub"):
                            used = variant
                            try:
                                fn = lambda: binding.pw_conv_i8(x, wp, cout, rq, y=y, variant=used)
                                fn()
                            except binding.PromError:
                                used = "auto"
                                fn = lambda: binding.pw_conv_i8(x, wp, cout, rq, y=y, variant=used)
                                fn()
                            iters = 5 if variant == "addsub" else 10
                            med, mn = cold_time_us(torch, fn, flush, iters=iters, warm=1)
                            same_as_naive = bool(torch.equal(y, y_ref))
                            rec = {"m": m, "k": cin, "n": cout, "zero_frac": z, "variant": variant,
                                   "ran_as": used, "us": round(med, 2),
                                   "gops": round(o / med / 1e3, 1), "gbs": round(b / med / 1e3, 1),
                                   "roof_us": round(roof, 2), "frac": round(roof / med, 4),
                                   "bound": "tensor" if o / p_i8 > b / bw else "hbm",
                                   "adds": m * nnz, "parity_vs_naive_whole": same_as_naive}
                            ok = same_as_naive
                            if want is not None:
                                rec["parity_vs_oracle_rows"] = bool(torch.equal(y[rows_d], want)) and naive_ok
                                rec["oracle_rows"] = int(rows.numel())
                                ok = ok and rec["parity_vs_oracle_rows"]
                            rec["parity"] = ok
                            bad += 0 if ok else 1
                            f.write(json.dumps(rec) + "\n")
                            f.flush()
                            n += 1
                    del y, y_ref
                del x
    st = binding.last_device_status()
    print(json.dumps({"sweep_points": n, "parity_failures": bad, "device_status": st, "file": args.sweep}),
          flush=True)
    return 0 if st == binding.PROM_OK and bad == 0 else 1


def run_single(args):
    """One single layer M,K,N[,variant[,zero_frac]] launched a few times (for profiler captures);
    variant tc_prepared times prom_pw_conv_i8_prepared on operands prepared once."""
    import torch
    from paper_2505_03254_b200 import binding, build, synth
    torch.cuda.set_device(0)
    build.build()
    binding.lib()
    parts = args.single.split(",")
    m, cin, cout = int(parts[0]), int(parts[1]), int(parts[2])
    variant = parts[3] if len(parts) > 3 else "auto"
    z = float(parts[4]) if len(parts) > 4 else 0.5
    pk = peaks()
    bw, p_i8 = pk["hbm_gbs"] * 1e9, i8_peak_probe(torch, binding)["tops_burst"] * 1e12
    seed = synth.BASE_SEED + 2
    x = synth.act_post_relu6(seed, (m, cin), device="cuda")
    lay = synth.make_layer(seed, cin, cout, z, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
    y = torch.empty((m, cout), dtype=torch.int8, device="cuda")
    flush = torch.empty((FLUSH_BYTES,), dtype=torch.uint8, device="cuda")
    if variant == "tc_prepared":
        prep = binding.pw_prepare(m, cin, wp, cout, rq)
        fn = lambda: binding.pw_conv_i8_prepared(x, cout, prep, y=y)
    else:
        fn = lambda: binding.pw_conv_i8(x, wp, cout, rq, y=y, variant=variant)
    med, mn = cold_time_us(torch, fn, flush, iters=max(1, args.steps), warm=max(1, args.warmup))
    b, o = layer_bytes(m, cin, cout), layer_ops(m, cin, cout)
    roof = max(b / bw, o / p_i8) * 1e6
    st = binding.last_device_status()
    print(json.dumps({"single": [m, cin, cout], "variant": variant, "zero_frac": z, "us": med,
                      "us_min": mn, "gbs": b / med / 1e3, "gops": o / med / 1e3, "roof_us": roof,
                      "frac": roof / med, "device_status": st}), flush=True)
    return 0 if st == binding.PROM_OK else 1


def run_widths(args):
    """The chained sequence at other width multipliers (Section 5 sweeps 0.75x-2.0x): step
    time, throughput and fraction of the summed per-layer roofline, each checked against the
    CPU oracle on one image.  One JSON object; not the headline line."""
    import torch
    from paper_2505_03254_b200 import binding, build, synth
    from oracle import prom_oracle
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    prom_oracle.build()
    binding.lib()
    pk = peaks()
    p_i8 = i8_peak_probe(torch, binding)["tops_burst"] * 1e12
    bw = pk["hbm_gbs"] * 1e9
    seed = synth.BASE_SEED + 3
    rows = []
    for width in [float(v) for v in args.widths.split(",")]:
        table, host, dev = build_network(seed, synth, binding, "cuda", width=width)
        seq = binding.LayerSeq(dev)
        c0, c1 = table[0].cin, table[-1].cout
        x0 = synth.act_post_relu6(seed, (BATCH, 112, 112, c0), device="cuda")
        ws = torch.empty((seq.workspace_bytes(BATCH, 112, 112),), dtype=torch.uint8, device="cuda")
        y = torch.empty((BATCH, 7, 7, c1), dtype=torch.int8, device="cuda")
        side = torch.cuda.Stream()
        torch.cuda.synchronize()          # the inputs were made on the default stream
        with torch.cuda.stream(side):
            binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
        for _ in range(5):
            graph.replay()
        steps = min(args.steps, 300)
        ms = time_region(torch, graph.replay, steps, False) / steps
        want = prom_oracle.layer_seq(host, x0[:1].cpu().numpy())
        ok = bool((y[:1].cpu().numpy() == want).all()) and binding.last_device_status() == binding.PROM_OK
        roof = sum(max(layer_bytes(BATCH * l.h * l.w, l.cin, l.cout) / bw,
                       layer_ops(BATCH * l.h * l.w, l.cin, l.cout) / p_i8) for l in table) * 1e6
        rows.append({"width": width, "ms_per_step": round(ms, 4), "images_per_s": round(BATCH / ms * 1e3, 1),
                     "weights": sum(l.cin * l.cout for l in table), "step_roofline_us": round(roof, 1),
                     "frac": round(roof / (ms * 1e3), 3), "parity_image_0": ok})
        del graph, ws, x0, y
    print(json.dumps({"widths": rows, "batch": BATCH, "unit": UNIT, "data": "synthetic"}))
    return 0 if all(r["parity_image_0"] for r in rows) else 1


def run_aux(args):
    """One of the legs that are off the timed step, alone (for profiling): act_quantizer,
    dynamic_layer or depthwise."""
    import torch
    from paper_2505_03254_b200 import binding, build, synth
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    build.build()
    binding.lib()
    bw = peaks()["hbm_gbs"] * 1e9
    if args.aux == "i8_peak":
        sampler = ClockSampler(0)
        sampler.start()
        out = i8_peak_probe(torch, binding, sustained_s=2.0)
        sampler.stop()
        pk = peaks()
        out["clocks"] = sampler.summary()
        out["two_x_measured_bf16_tops"] = INT8_OVER_BF16 * pk["bf16_tflops"]
        out["two_x_measured_bf16_sustained_tops"] = INT8_OVER_BF16 * pk["bf16_tflops_sustained"]
        out["nominal_tops"] = NOMINAL_I8_TOPS
    elif args.aux == "alu_rate":
        out = alu_rate_probe(torch, binding)
    elif args.aux == "write_bw":
        out = write_bandwidth_probe(torch)
    elif args.aux == "mma_beside":
        out = mma_beside_probe(torch, binding)
    elif args.aux == "mma_issue":
        out = mma_issue_probe(torch, binding)
    elif args.aux == "l2_copy":
        out = l2_copy_probe(torch, binding)
    elif args.aux == "depth_first":
        out = depth_first_timing(torch, binding, synth)
    elif args.aux == "act_quantizer":
        out = act_quantizer_timing(torch, binding, bw)
    elif args.aux == "dynamic_layer":
        out = dynamic_layer_timing(torch, binding, synth, bw)
    elif args.aux == "body":
        out = {"plain": body_with_depthwise_timing(torch, binding, synth, bw),
               "skips": body_with_depthwise_timing(torch, binding, synth, bw, skips=True)}
    else:
        out = depthwise_timing(torch, binding, bw)
    print(json.dumps({"aux": args.aux, "result": out, "device_status": binding.last_device_status()}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "stub"])
    ap.add_argument("--variant", default="auto", choices=["auto", "tc", "naive"])
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of a CUDA graph")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--no-detail", action="store_true", help="skip per-layer and single-layer timing")
    ap.add_argument("--sweep", default=None, help="write the single-layer sweep to this file")
    ap.add_argument("--single", default=None, help="M,K,N[,variant[,zero_frac]]: time one layer")
    ap.add_argument("--aux", default=None, choices=["act_quantizer", "dynamic_layer", "depthwise", "body", "i8_peak", "alu_rate", "depth_first", "mma_issue", "l2_copy", "write_bw", "mma_beside"],
                    help="run one of the legs that are off the timed step, alone")
    ap.add_argument("--widths", default=None, help="comma-separated width multipliers: time the sequence at each")
    ap.add_argument("--sweep-small", action="store_true", help="sweep without the largest M")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    plain_leg = not (args.widths or args.aux or args.single or args.sweep)
    if args.gpus > 1 and plain_leg and "RANK" not in os.environ and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args, sys.argv[1:])
    if args.impl == "stub":
        return run_stub(args)
    if args.widths:
        return run_widths(args)
    if args.aux:
        return run_aux(args)
    if args.single:
        return run_single(args)
    if args.sweep:
        return run_sweep(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
