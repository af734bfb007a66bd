#!/usr/bin/env python
"""Benchmark of the PeRQ online path (permute -> block Hadamard -> INT4/MXFP4) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one perq_rotate_quantize call over the headline workload (Llama-3-8B-shaped
hidden activations, T=16384 x d=4096 bf16, block Hadamard b=32, INT4 per-token scale).
`value` is the effective bandwidth: algorithmic bytes (bf16 row in + packed codes +
scales out) per second, inputs resident in HBM.  Prints ONE JSON line (rank 0).

The other variants of the same workload (b in {16,32,128,4096} x {INT4, MXFP4}) and the
calibration statistic are timed after the K steps and reported under "sweep".
`--impl reference` times the CPU oracle instead (a deliberately plain fp64 program).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "rotate_quantize_effective_hbm_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# headline workload
T_HEAD, D_HEAD, B_HEAD, FMT_HEAD, GROUP_HEAD = 16384, 4096, 32, "int4", 0
ORACLE_FMT = {"int4": 0, "mxfp4": 1, "fp4": 3}     # format numbers of oracle/perq_oracle.c

# DRAM traffic of one launch of the headline kernel (dram__bytes_read.sum + dram__bytes_write.sum from an ncu
# capture) is kept in a small tracked file together with the names and a hash of the sources that kernel is compiled from;
# when the sources have changed since, the bench reports no traffic figure.
TRAFFIC_FILE = os.path.join(ROOT, "paper_2601_22347_b200", "ncu_traffic.json")


def kernel_sources_hash(names):
    """SHA-256 over the named files of csrc/ (the sources a captured kernel is compiled from)."""
    import hashlib
    csrc = os.path.join(ROOT, "paper_2601_22347_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(names):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()


def captured_traffic(fmt):
    """Bytes per launch from the last ncu capture of this format's headline kernel, or None if there is none
    for that kernel's sources as they are now."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(fmt)
        if rec is None or rec.get("sources_sha256") != kernel_sources_hash(rec["sources"]):
            return None
        return rec.get("dram_bytes_per_launch")
    except Exception:
        return None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.12)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return out
        sm, mx, reasons = [], [], set()
        for line in text.strip().splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def bytes_per_token(d, fmt, group):
    from paper_2601_22347_b200.roofline import algorithmic_bytes_per_token
    return algorithmic_bytes_per_token(d, fmt, group)


# ------------------------------------------------------------------------------ reference arm (CPU oracle)

def run_reference(args):
    """Times the oracle, as it stands, on the host cores; each step is a bounded row sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np
    from oracle import perq_oracle
    from paper_2601_22347_b200 import inputs
    perq_oracle.build()
    fmt = ORACLE_FMT[FMT_HEAD]
    w = inputs.config4(T=2048, b=B_HEAD, fmt=FMT_HEAD)
    # bounded sample: as many rows per step (16 .. 2048) as keep the K steps within about a minute
    perq_oracle.rotate_quantize(w.x[:256], None, w.b, fmt, w.group)
    t0 = time.perf_counter()
    perq_oracle.rotate_quantize(w.x[:256], None, w.b, fmt, w.group)
    per_row = (time.perf_counter() - t0) / 256
    rows = int(min(2048, max(16, 60.0 / (max(1, args.steps) * per_row))))
    w.x = np.ascontiguousarray(w.x[:rows])
    for _ in range(max(1, min(args.warmup, 2))):
        perq_oracle.rotate_quantize(w.x, None, w.b, fmt, w.group)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        perq_oracle.rotate_quantize(w.x, None, w.b, fmt, w.group)
    dt = (time.perf_counter() - t0) / args.steps
    bpt = bytes_per_token(D_HEAD, FMT_HEAD, GROUP_HEAD)
    value = rows * bpt / dt / 1e9
    sample = "%d of %d rows per step (rows are independent)" % (rows, T_HEAD)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg4 Llama-3-8B hidden: T=%d d=%d bf16 Laplace+4 outlier channels, b=%d, %s"
                               % (T_HEAD, D_HEAD, B_HEAD, FMT_HEAD), "sample": sample},
        "mtokens_per_s": rows / dt / 1e6,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": perq_oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------ CUDA arm

def main():
    global FMT_HEAD, GROUP_HEAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="perq", choices=["perq", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-variant sweep after the timed steps")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fmt", default=FMT_HEAD, choices=["int4", "mxfp4", "fp4"],
                    help="format of the timed step (default: the headline, INT4 with a per-token scale)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    FMT_HEAD, GROUP_HEAD = args.fmt, (32 if args.fmt == "mxfp4" else 0)
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly with --gpus N: become the launcher of N ranks (one per GPU) of this same command
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        return subprocess.call(cmd)

    import numpy as np
    import torch
    from paper_2601_22347_b200 import binding as B, inputs, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        sys.stderr.write("bench.py: --gpus %d but WORLD_SIZE is %d\n" % (args.gpus, world))
        return 2
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.load()

    # Every rank holds the same-shaped workload with its own seed: rows are independent, so the
    # path shards over T with no data-path collective (weak scaling).
    w = inputs.config4(T=T_HEAD, b=B_HEAD, fmt=FMT_HEAD, variant=rank % 10)
    fmt = B.FMT_BY_NAME[FMT_HEAD]
    RING = 4   # 4 x 134 MB of inputs: every call reads rows that are not in the 126 MB L2
    base = torch.from_numpy(w.x.view(np.int16).copy()).cuda().view(torch.bfloat16)
    xs = [base] + [torch.roll(base, shifts=17 * (i + 1), dims=0).contiguous() for i in range(RING - 1)]
    outs = [B.alloc_outputs(T_HEAD, D_HEAD, fmt, GROUP_HEAD, base.device) for _ in range(RING)]
    bpt = bytes_per_token(D_HEAD, FMT_HEAD, GROUP_HEAD)
    bytes_per_step = bpt * T_HEAD

    def step(i):
        k = i % RING
        B.perq_rotate_quantize(xs[k], None, B_HEAD, fmt, GROUP_HEAD, out_codes=outs[k][0], out_scales=outs[k][1])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        # nvidia-smi needs a moment to start sampling: keep the GPU under the same load meanwhile (untimed)
        sampler.start()
        t_end = time.perf_counter() + 0.4
        i = 0
        while time.perf_counter() < t_end:
            step(i)
            i += 1
            if i % 256 == 0:
                torch.cuda.synchronize()
    barrier()
    # One event before the K steps and one after them (the step is a single kernel, so the average launch
    # duration is their distance over K), plus a few in between to show the spread.  An event after every
    # launch would itself add a few microseconds to each 40 us step.
    marks = sorted(set([0, args.steps] + [args.steps * k // 8 for k in range(1, 8)]))
    ev = {m: torch.cuda.Event(enable_timing=True) for m in marks}
    # a few untimed launches are queued first, so that the first event is recorded behind running work and a
    # short run does not time the start of the queue
    LEAD = 8
    for i in range(LEAD):
        step(i)
    ev[0].record()
    for i in range(args.steps):
        step(LEAD + i)
        if i + 1 in ev:
            ev[i + 1].record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = ev[0].elapsed_time(ev[args.steps])
    local_ms = total_ms
    per_launch_ms = [ev[a].elapsed_time(ev[b]) / (b - a) for a, b in zip(marks[:-1], marks[1:])]
    total_ms = sharding.max_over_ranks(total_ms, device="cuda")
    ms_per_step = total_ms / args.steps
    value = world * bytes_per_step / (ms_per_step * 1e-3) / 1e9

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    xh = torch.from_numpy(w.x.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    ch = torch.empty((T_HEAD, D_HEAD // 2), dtype=torch.uint8).pin_memory()
    sh = (torch.empty((T_HEAD, D_HEAD // 32), dtype=torch.uint8) if FMT_HEAD == "mxfp4"
          else torch.empty((T_HEAD, 1), dtype=torch.float32)).pin_memory()
    ws = torch.empty(B.perq_host_workspace_bytes(T_HEAD, D_HEAD, fmt, GROUP_HEAD), dtype=torch.uint8, device="cuda")
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        B.perq_rotate_quantize_host(xh, None, B_HEAD, fmt, GROUP_HEAD, ch, sh, ws)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        B.perq_rotate_quantize_host(xh, None, B_HEAD, fmt, GROUP_HEAD, ch, sh, ws)   # synchronises its stream
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    e2e_s = sharding.max_over_ranks(e2e_s, device="cuda")
    e2e = {"value": world * bytes_per_step / e2e_s / 1e9, "unit": UNIT,
           "h2d_bytes_per_step": int(xh.numel() * 2), "d2h_bytes_per_step": int(ch.numel() + sh.numel() * sh.element_size()),
           "ms_per_step": e2e_s * 1e3, "api": "perq_rotate_quantize_host"}
    del ws

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peak()
    launch_ms = local_ms / args.steps          # this rank's K launches between its two events
    achieved = bytes_per_step / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": "of " + peak_kind, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "traffic": captured_traffic(FMT_HEAD),
                "algorithmic_bytes_per_launch": bytes_per_step, "kernel_ms": launch_ms,
                "kernel_ms_by_eighth_of_the_run": [round(v, 5) for v in per_launch_ms]}

    sweep = []
    check_rows = None
    if not args.no_cpu_baseline:
        # beside every timed variant: a few rows of the last call's outputs against the oracle (part of the CPU leg)
        from oracle import perq_oracle
        perq_oracle.build()
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        from parity import compare_quantized

        def check_rows(x_dev, perm, b, f, grp, codes, scales, n=16):
            T = x_dev.shape[0]
            rows = np.unique(np.linspace(0, T - 1, num=min(n, T)).astype(np.int64))
            rt = torch.from_numpy(rows).to(x_dev.device)
            bits = x_dev[rt].view(torch.int16).cpu().numpy().view(np.uint16)
            ora = perq_oracle.rotate_quantize(bits, perm, b, B.FMT_BY_NAME[f], grp, want_pre=True)
            rep = compare_quantized(f, codes[rt].cpu().numpy(), scales[rt].cpu().numpy(), ora)
            return {"parity_rows_checked": int(rows.size), "tie_window_exemptions": rep["code_mismatch_exempt"]}

    if not args.no_sweep:
        def time_calls(fn, n=30, warm=5):
            for i in range(warm):
                fn(i)
            torch.cuda.synchronize()
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n):
                fn(i)
            b_.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b_) / n

        for f in ("int4", "mxfp4", "fp4", "int4_asym"):
            fcode = B.FMT_BY_NAME[f]
            grp = 32 if f == "mxfp4" else 0
            o = [B.alloc_outputs(T_HEAD, D_HEAD, fcode, grp, base.device) for _ in range(RING)]
            for bb in ((16, 32, 128, 4096) if f in ("int4", "mxfp4") else (32,)):
                ms = time_calls(lambda i: B.perq_rotate_quantize(xs[i % RING], None, bb, fcode, grp,
                                                                 out_codes=o[i % RING][0], out_scales=o[i % RING][1]))
                by = bytes_per_token(D_HEAD, f, grp) * T_HEAD
                gbs = by / (ms * 1e-3) / 1e9
                row = {"call": "perq_rotate_quantize", "T": T_HEAD, "d": D_HEAD, "b": bb, "fmt": f, "group": grp,
                       "ms": ms, "GB/s": gbs, "frac_of_" + peak_kind: gbs / peak,
                       "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "Mtokens/s": T_HEAD / ms / 1e3}
                if check_rows is not None:
                    B.perq_rotate_quantize(xs[0], None, bb, fcode, grp, out_codes=o[0][0], out_scales=o[0][1])
                    torch.cuda.synchronize()
                    row.update(check_rows(xs[0], None, bb, f, grp, o[0][0], o[0][1]))
                sweep.append(row)
            del o
        # the calibration statistic on the MLP down-projection shape (T=4096 x d=8192, b=32)
        w3 = inputs.config3(T=4096)
        x3 = [torch.from_numpy(w3.x.view(np.int16).copy()).cuda().view(torch.bfloat16)]
        x3 += [torch.roll(x3[0], shifts=5 * (i + 1), dims=0).contiguous() for i in range(RING - 1)]
        wsb = torch.empty(B.perq_block_l1_stats_workspace_bytes(4096, 8192, 32), dtype=torch.uint8, device="cuda")
        ms = time_calls(lambda i: B.perq_block_l1_stats(x3[i % RING], None, 32, workspace=wsb))
        by = 4096 * 8192 * 2
        sweep.append({"call": "perq_block_l1_stats", "T": 4096, "d": 8192, "b": 32, "ms": ms,
                      "GB/s": by / (ms * 1e-3) / 1e9, "frac_of_" + peak_kind: by / (ms * 1e-3) / 1e9 / peak})
        del xs, outs, base

        # the other workloads, with their permutations (cold inputs: rings larger than L2)
        def time_workload(name, bits, perm, b, f, grp):
            T, d = bits.shape
            fcode = B.FMT_BY_NAME[f]
            ring = max(2, int(300e6 // max(1, T * d * 2)) + 1)
            ring = min(ring, 64)
            x0 = torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)
            xr = [x0] + [torch.roll(x0, shifts=3 * (i + 1), dims=0).contiguous() if T > 1 else x0.clone()
                         for i in range(ring - 1)]
            orr = [B.alloc_outputs(T, d, fcode, grp, x0.device) for _ in range(ring)]
            pd = None if perm is None else torch.from_numpy(perm).cuda()
            ms = time_calls(lambda i: B.perq_rotate_quantize(xr[i % ring], pd, b, fcode, grp,
                                                             out_codes=orr[i % ring][0], out_scales=orr[i % ring][1]))
            by = bytes_per_token(d, f, grp) * T
            gbs = by / (ms * 1e-3) / 1e9
            row = {"call": "perq_rotate_quantize", "workload": name, "T": T, "d": d, "b": b, "fmt": f, "group": grp,
                   "perm": perm is not None, "us": ms * 1e3, "GB/s": gbs, "frac_of_" + peak_kind: gbs / peak,
                   "Mtokens/s": T / ms / 1e3}
            if by < 64e6:
                # small calls are bound by the host's launch rate when issued one by one from Python: the same
                # calls replayed from a CUDA graph (50 per graph) give the device-side time per call
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(50):
                        B.perq_rotate_quantize(xr[i % ring], pd, b, fcode, grp, out_codes=orr[i % ring][0],
                                               out_scales=orr[i % ring][1], stream=torch.cuda.current_stream())
                gms = time_calls(lambda i: graph.replay(), n=10, warm=2) / 50
                row["us_graph_replay"] = gms * 1e3
                row["GB/s_graph_replay"] = by / (gms * 1e-3) / 1e9
                del graph
            if check_rows is not None:
                B.perq_rotate_quantize(xr[0], pd, b, fcode, grp, out_codes=orr[0][0], out_scales=orr[0][1])
                torch.cuda.synchronize()
                row.update(check_rows(xr[0], perm, b, f, grp, orr[0][0], orr[0][1]))
            sweep.append(row)

        # the gated-activation entry point on the MLP down-projection shape: two bf16 projections in, h never stored
        rng3 = np.random.default_rng(inputs.SEED_BASE + 33)
        gate_bits = inputs.f32_to_bf16_bits((rng3.standard_normal((4096, 8192)) * 2.0).astype(np.float32))
        up_bits = inputs.f32_to_bf16_bits(rng3.standard_normal((4096, 8192)).astype(np.float32))
        gates = [torch.from_numpy(gate_bits.view(np.int16).copy()).cuda().view(torch.bfloat16)]
        ups = [torch.from_numpy(up_bits.view(np.int16).copy()).cuda().view(torch.bfloat16)]
        for i in range(2):
            gates.append(torch.roll(gates[0], shifts=5 * (i + 1), dims=0).contiguous())
            ups.append(torch.roll(ups[0], shifts=5 * (i + 1), dims=0).contiguous())
        og = [B.alloc_outputs(4096, 8192, B.PERQ_FMT_MXFP4, 32, gates[0].device) for _ in range(3)]
        ms = time_calls(lambda i: B.perq_swiglu_rotate_quantize(gates[i % 3], ups[i % 3], None, 32, B.PERQ_FMT_MXFP4, 32,
                                                                out_codes=og[i % 3][0], out_scales=og[i % 3][1]))
        by = (2 * 2 * 8192 + 8192 // 2 + 8192 // 32) * 4096
        row = {"call": "perq_swiglu_rotate_quantize", "T": 4096, "d": 8192, "b": 32, "fmt": "mxfp4", "group": 32, "ms": ms,
               "bytes": by, "GB/s": by / (ms * 1e-3) / 1e9, "frac_of_" + peak_kind: by / (ms * 1e-3) / 1e9 / peak}
        if check_rows is not None:
            B.perq_swiglu_rotate_quantize(gates[0], ups[0], None, 32, B.PERQ_FMT_MXFP4, 32, out_codes=og[0][0], out_scales=og[0][1])
            torch.cuda.synchronize()
            rows16 = np.unique(np.linspace(0, 4095, num=16).astype(np.int64))
            hb = perq_oracle.swiglu(gate_bits[rows16], up_bits[rows16])
            ora = perq_oracle.rotate_quantize(hb, None, 32, B.PERQ_FMT_MXFP4, 32, want_pre=True)
            rt = torch.from_numpy(rows16).cuda()
            rep = compare_quantized("mxfp4", og[0][0][rt].cpu().numpy(), og[0][1][rt].cpu().numpy(), ora)
            row.update({"parity_rows_checked": int(rows16.size), "tie_window_exemptions": rep["code_mismatch_exempt"]})
        sweep.append(row)
        del gates, ups, og

        w1 = inputs.config1()
        time_workload("cfg1", w1.x, None, 16, "int4", 0)
        w2 = inputs.config2(T=4096, b=32)
        time_workload("cfg2", w2.x, w2.perm, 32, "int4", 128)
        chan, _, _ = B.perq_block_l1_stats(x3[0], None, 32, want=("chan",), workspace=wsb)
        torch.cuda.synchronize()
        # Algorithm 1 on the device (sequential greedy: a latency figure, not a bandwidth one), checked against the host one
        pws = torch.empty(8192 * 4, dtype=torch.uint8, device="cuda")
        pdev = torch.empty(8192, dtype=torch.int32, device="cuda")
        ms = time_calls(lambda i: B.perq_massdiff_perm_device(chan, 32, perm=pdev, workspace=pws), n=5, warm=1)
        phost = B.perq_massdiff_perm(chan.cpu().numpy(), 32)
        sweep.append({"call": "perq_massdiff_perm_device", "d": 8192, "b": 32, "ms": ms,
                      "equals_host_permutation": bool(np.array_equal(pdev.cpu().numpy(), phost))})
        time_workload("cfg3 (MassDiff permutation)", w3.x, phost, 32, "mxfp4", 32)
        del x3
        for T5 in (1, 16, 128, 1024, 16384):
            w5 = inputs.config5(T=T5, b=32)
            time_workload("cfg5", w5.x, w5.perm, 32, "int4", 128)
        # full-vector rotation of a width that is not a power of two (14336 = 2^9 x 28, general kernel)
        w5 = inputs.config5(T=1024, b=32)
        time_workload("cfg5 width, full-vector 2^9 x 28", w5.x, None, 14336, "int4", 0)
        time_workload("cfg5 width, full-vector 2^9 x 28", w5.x, None, 14336, "mxfp4", 32)

    cpu_baseline = None
    if not args.no_cpu_baseline:
        rows = 4096
        wb = inputs.config4(T=rows, b=B_HEAD, fmt=FMT_HEAD)
        perq_oracle.rotate_quantize(wb.x[:256], None, B_HEAD, ORACLE_FMT[FMT_HEAD], GROUP_HEAD)
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            perq_oracle.rotate_quantize(wb.x, None, B_HEAD, ORACLE_FMT[FMT_HEAD], GROUP_HEAD)
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        cpu_baseline = {"value": rows * bpt / dt / 1e9, "unit": UNIT, "cores": perq_oracle.num_threads(),
                        "kind": "oracle", "mtokens_per_s": rows / dt / 1e6,
                        "sample": "%d of %d rows of the same workload, repeated for ~10 s (%d passes)" % (rows, T_HEAD, reps)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "cfg4 Llama-3-8B hidden: T=%d d=%d bf16 Laplace(0,1)+4 outlier channels x200, no perm, "
                               "block Hadamard b=%d, %s" % (T_HEAD, D_HEAD, B_HEAD, {"int4": "INT4 per-token absmax scale",
                               "mxfp4": "MXFP4 (E2M1 + E8M0 per 32)", "fp4": "FP4 (E2M1) per-token scale"}[FMT_HEAD]),
                   "per_gpu_tokens": T_HEAD, "l2": "ring of %d input sets, each 134 MB > 126 MB L2" % RING},
        "mtokens_per_s": world * T_HEAD / ms_per_step / 1e3,
        "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
        "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps,
        "roofline": roofline, "cpu_baseline": cpu_baseline, "sweep": sweep,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
